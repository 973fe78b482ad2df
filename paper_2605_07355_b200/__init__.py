"""B200-native Temporal Token Fusion (arXiv 2605.07355, Sec. 3): the pre-LLM token-compression pass as a
C-ABI CUDA library (libttf_b200.so, include/ttf.h) with a thin binding.  Importing the package loads nothing;
the shared library is opened on the first call."""
from . import clips  # noqa: F401  (seeded synthetic clips; no method arithmetic)


def __getattr__(name):
    if name.startswith(("ttf_", "TTF_")) or name in ("TTFError", "lib", "LIB_PATH", "EXPORTS", "KERNEL_KINDS", "TTF_STATIC_SCRATCH_BYTES", "TTF_DTYPE_F32", "TTF_DTYPE_BF16"):
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
