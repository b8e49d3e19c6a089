"""Hydra speculative-decode step for one B200 (sm_100a): thin Python binding over libhydra's C ABI.

Every step of the path runs in the library's CUDA kernels; this package only marshals arguments.
torch provides device memory and streams.  There is no CPU fallback: touching any binding name raises
ImportError if the shared library has not been built (python -m paper_2402_05109_b200.build).
"""
_BINDING_NAMES = ("Hydra", "HydraError", "lib", "gemm", "gemm_noalloc", "tree_attention", "gemm_bounded_wait_probe", "LIB_PATH", "BUF")


def __getattr__(name):
    if name in _BINDING_NAMES:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
