"""Fused Slide Attention forward (arXiv 2304.04237) for NVIDIA B200: Python binding of the
C-ABI library in csrc/.  See include/slide_attn.h for the contract."""
from . import binding  # noqa: F401
from .binding import (BF16, ERR_ALIGNMENT, ERR_ALLOC, ERR_ARCH, ERR_CUDA, ERR_INVALID_ARG,  # noqa: F401
                      ERR_TIMEOUT, ERR_TOO_LARGE, ERR_NOT_FIXED_SHIFT, ERR_UNSUPPORTED, F32, OK, VARIANT_AUTO, VARIANT_DIRECT,
                      VARIANT_MMA, VARIANT_UMMA_TS, VARIANT_STRIP, VARIANT_TILE, VARIANT_MMA_WIDE, SlideAttnError, slide_attn_create,
                      slide_attn_destroy, slide_attn_forward, slide_attn_backward, slide_attn_forward_host, slide_attn_forward_noalloc,
                      slide_attn_get_variant, slide_attn_launches_per_forward,
                      slide_attn_profile_begin, slide_attn_profile_end,
                      slide_attn_query_status, slide_attn_set_variant, slide_attn_status_string,
                      slide_attn_set_fixed_shift, slide_attn_detect_fixed_shift,
                      slide_attn_project, slide_attn_block_forward)
