"""Fused MLP-Adam cross-validation on B200: thin binding over the C-ABI library.

The compute lives in ``libbbo_mlp_cv.so`` (CUDA, sm_100a).  Importing this
package does not load it; the first call into :mod:`.binding` does, and fails
loudly if the library has not been built.  There is no CPU fallback.
"""
__all__ = ["binding", "workloads"]
