// Placeholder entry points until the fused forward lands.
#include "efq_common.cuh"
extern "C" size_t efq_attention_workspace_bytes(int, int, int, int64_t, int64_t, int) { return 0; }
extern "C" efq_status_t efq_attention_fwd(const void*, const void*, const void*, float*, int, int, int, int64_t, int64_t, int, int, float, const efq_params_t*, void*, size_t, const efq_debug_t*, void*) { return EFQ_ERR_UNSUPPORTED; }
extern "C" efq_status_t exp_then_quantize_attention_fwd(const void*, const void*, const void*, float*, int, int, int, int64_t, int64_t, int, int, float, int, void*, size_t, const efq_debug_t*, void*) { return EFQ_ERR_UNSUPPORTED; }
extern "C" efq_status_t efq_attention_fwd_host(const void*, const void*, const void*, float*, void*, void*, void*, float*, int, int, int, int64_t, int64_t, int, int, float, int, const efq_params_t*, void*, size_t, void*) { return EFQ_ERR_UNSUPPORTED; }
extern "C" efq_status_t efq_poll_status(void*, void*) { return EFQ_ERR_UNSUPPORTED; }
extern "C" efq_status_t efq_fp4_mma_peak_probe(uint32_t*, int, int, double*, void*) { return EFQ_ERR_UNSUPPORTED; }
