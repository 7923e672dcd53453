"""B200-native Gumbel-max list sampling (arXiv 2506.05632): Python binding of libgls.

The functions here only marshal arguments (torch tensors -> raw device pointers, strides in
elements) into the C ABI declared in include/gls.h; every step of the method runs in the CUDA
kernels of csrc/.  There is no CPU fallback: if libgls.so cannot be loaded the calls raise.

    draft_sample(logits, ...)                 Algorithm 1 third step / Algorithm 2 draft loop
    target_sample_verify(logits, tokens, ...) Algorithm 2 verification
    draft_verify(draft, target, ...)          both of the above in one call (one sweep launch)
    compress_select(enc, dec, bins, ...)      Sec. 5.1 encoder / decoder index selection
    compress_gaussian(u, a, t, bins, ...)     the same from the source: Appendix C weights computed in the kernels
"""
from .binding import (  # noqa: F401
    COMBINE_ACTIVE, COMBINE_ALL, NO_BONUS, VERIFY_ALL_ROWS, VERIFY_ACTIVE_ROWS, VERIFY_FIRST_PHASE,
    VERIFY_REST, VERIFY_THREE_PHASES, NOISE_SHARED_ACROSS_K,
    DEV_EMPTY_SUPPORT, GlsError,
    build, copy_rows_to_device, debug_bounds, compress_gaussian, compress_gaussian_workspace_bytes, compress_select, draft_sample, draft_sample_sparse, draft_sample_static,
    draft_sample_topm, draft_verify, draft_verify_workspace_bytes, lib_path, load,
    static_scratch_bytes, status_string, target_sample_verify, target_sample_verify_sparse,
    target_sample_verify_topm, topm_workspace_bytes, verify_phases, verify_walk, version, workspace_bytes)
