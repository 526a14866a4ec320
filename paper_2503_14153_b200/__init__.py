"""B200-native draft-and-verify decode loop (Medusa-style speculative decoding, Sec. III-B).

The work is done by hand-written sm_100a kernels behind a C ABI (include/spec_decode.h);
this package is the thin ctypes binding plus the candidate-tree generator. Importing the
package does not load the shared library; the first call that needs it does, and fails
loudly if it has not been built.
"""
from .tree import build_tree, chain_tree  # noqa: F401
from .binding import (SpecDecoder, SpecError, load_library, library_path, spec_op_linear, spec_op_linear_static, spec_build_labels,  # noqa: F401
                      upload_weights, FLAG_KEEP_LOGITS, FLAG_SIMPLE_KERNELS, FLAG_PACKED_WEIGHTS,
                      spec_pack_weight, pack_linear_weights)
