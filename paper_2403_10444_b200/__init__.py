"""B200-native batched draft verification for speculative decoding (arXiv 2403.10444).

The product is the C-ABI library ``libbv_b200.so`` (see ``include/bv.h``); this
package is its thin Python binding.  Importing the package does not load the
library; calling any entry point does, and raises if it has not been built.
"""
from .binding import (bv_verify, tv_verify, bv_verify_ex, tv_verify_ex, bv_verify_host,
                      tv_verify_host, bv_verify_noalloc, bv_verify_lse, tv_verify_lse, gbv_verify, gbv_verify_ex, bv_verify_probs, tv_verify_probs, bv_sample_draft, bv_draft_chain, bv_release, bv_set_option, bv_stream_status, bv_last_launch_count, bv_last_kernel, bv_status_string,
                      bv_version, load_library, BVError, DTYPE_F32, DTYPE_BF16, EXPORTS)

__all__ = ["bv_verify", "tv_verify", "bv_verify_ex", "tv_verify_ex", "bv_verify_host",
           "tv_verify_host", "bv_verify_noalloc", "bv_verify_lse", "tv_verify_lse", "gbv_verify", "gbv_verify_ex", "bv_verify_probs", "tv_verify_probs", "bv_sample_draft", "bv_draft_chain", "bv_release", "bv_set_option", "bv_stream_status", "bv_last_launch_count", "bv_last_kernel", "bv_status_string",
           "bv_version", "load_library", "BVError", "DTYPE_F32", "DTYPE_BF16", "EXPORTS"]
