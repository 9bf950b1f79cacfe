"""B200-native PaSS (Parallel Speculative Sampling) decoder step.

The product is the C-ABI library built from ``csrc/`` (declared in
``include/pass.h``); this package is a thin ctypes binding with the same names.
"""
from .binding import (PassContext, PassError, load_library, LIB_PATH,  # noqa: F401
                      PASS_DBG_LOGITS, PASS_DBG_DRAFT_LOGITS, PASS_DBG_KV_LEN, PASS_DBG_N_DRAFT,
                      PASS_DBG_DRAFTS, PASS_DBG_PENDING, PASS_DBG_N_ACCEPTED, PASS_DBG_STATUS,
                      PASS_DBG_HIDDEN, PASS_DBG_FOOTPRINT, PASS_MAX_TOP_K, PASS_HOOK_GEMM_STUCK, PASS_HOOK_ATTN_STALE, PASS_HOOK_ATTN_LONG_FROM, PASS_HOOK_ATTN_STUCK, PASS_PROMPT_HI_LO, PASS_PROMPT_BF16, PASS_TRAIN_LA, PASS_TRAIN_GRAD)
