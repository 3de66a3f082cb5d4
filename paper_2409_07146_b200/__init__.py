"""B200-native Gated Slot Attention layer (arXiv 2409.07146): thin Python binding over
the C-ABI CUDA library ``libgsa.so`` built from ``csrc/``.

The binding only marshals arguments (device pointers of torch tensors, sizes, the
current CUDA stream); every step of the layer runs in the library's kernels.  There is
no CPU path: importing works without a GPU (so that the library's exports can be
checked), but every compute call needs CUDA tensors and raises otherwise.
"""
from .binding import (  # noqa: F401
    GsaError, Params, lib_path, load_library, exported_symbols,
    gsa_chunk_size, gsa_workspace_bytes, gsa_gate_cumsum, gsa_fwd, gsa_bwd, gsa_decode_step, gsa_tc_selftest,
    gsa_timing_begin, gsa_timing_end, gsa_fwd_noalloc, gate_block, GSA_NOALLOC_MAX_WORKSPACE_BYTES,
    gsa_wait_selftest, gsa_release_streams, gsa_shard_states, gsa_shard_combine, gsa_out_norm_fwd, gsa_out_norm_bwd,
    gsa_dev_pair_scans,
)
