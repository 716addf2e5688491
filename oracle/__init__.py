"""CPU oracle for the EFQ-Softmax hot path (test infrastructure only).

Nothing in the product package imports this.  ``oracle.efq_oracle`` wraps the plain C
implementation (built on demand with gcc); ``oracle.efq_math`` is a double-precision
numpy evaluation of the paper's equations used to pin the C code.
"""
