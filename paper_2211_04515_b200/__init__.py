"""B200-native activation quantization path of QuantPipe (arXiv 2211.04515, Sec. 3):
statistics, ACIQ clip, directed search, quantize + bit-pack, unpack + dequantize, bit-width
selection.  The work is done by libquantpipe.so (hand-written sm_100a CUDA behind a C ABI,
declared in include/quantpipe.h); this package only marshals arguments."""
from .binding import *  # noqa: F401,F403
from .binding import Context, Controller, DSResult, QParams, QuantPipeError, Stats, load  # noqa: F401
