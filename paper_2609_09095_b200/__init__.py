"""B200-native (sm_100a) Ozaki Scheme II emulated-FP64 GEMM: thin Python binding over the
C-ABI library liboz_b200.so.  Every step of the method runs in the library's CUDA kernels; this
package only marshals arguments (torch tensors -> device pointers)."""
from .binding import *  # noqa: F401,F403
from .binding import __all__  # noqa: F401
