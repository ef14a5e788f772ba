"""B200 (sm_100a) implementation of the Polymorph multi-LoRA ViT forward path.

The product is the C-ABI library `libpolymorph.so` (see include/polymorph.h); `binding` is its thin
ctypes wrapper.  Importing this package does not load the library; `binding.load()` does and
raises if it has not been built.
"""
from . import binding  # noqa: F401
