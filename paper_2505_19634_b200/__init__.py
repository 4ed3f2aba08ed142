"""B200-native verify step of batched speculative decoding (attention + accept/resample).

Thin Python binding over the C-ABI library (include/tts.h).  Every step of the path runs in
the sm_100a kernels of libtts_b200.so; this package only marshals arguments.
"""
from .binding import (ATTN_AUTO, ATTN_SIMT, ATTN_TCGEN05, ATTN_TCGEN05_ROW_MAJOR, ATTN_TCGEN05_TOKEN_MAJOR, MASK_CAUSAL, MASK_TREE, OUT_BF16, OUT_FP32, LOGITS_BF16, LOGITS_FP32,
                      TtsConfig, TtsContext, TtsError, EXPORTED_SYMBOLS, library_path, load_library,
                      tts_confidence_max, tts_greedy_search, tts_grid_search, tts_majority_vote, tts_strerror,
                      tts_verify_attn_noalloc)

__all__ = ["ATTN_AUTO", "ATTN_SIMT", "ATTN_TCGEN05", "ATTN_TCGEN05_ROW_MAJOR", "ATTN_TCGEN05_TOKEN_MAJOR", "MASK_CAUSAL", "MASK_TREE", "OUT_BF16", "OUT_FP32", "LOGITS_BF16", "LOGITS_FP32",
           "TtsConfig", "TtsContext", "TtsError", "EXPORTED_SYMBOLS", "library_path", "load_library",
           "tts_confidence_max", "tts_greedy_search", "tts_grid_search", "tts_majority_vote", "tts_strerror", "tts_verify_attn_noalloc"]
