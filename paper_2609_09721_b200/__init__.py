"""B200-native EFQ-Softmax hot path: a C-ABI CUDA library (sm_100a) and a thin Python binding.

``paper_2609_09721_b200.binding`` exposes the library's entry points under the same names
(argument marshalling only; every step of the path runs in the CUDA kernels).
``paper_2609_09721_b200.inputs`` holds the seeded synthetic workloads.
"""

__all__ = ["binding", "inputs", "build"]
