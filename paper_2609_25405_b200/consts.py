"""Enumerations of the C ABI (mirrors include/hb.h); importable without the CUDA library."""
KIND_DECODE, KIND_PREFILL_CHUNK, KIND_EMBED_CHUNK = 0, 1, 2
POOL_NONE, POOL_MEAN, POOL_LAST, POOL_CLS, POOL_WMEAN, POOL_MAX = 0, 1, 2, 3, 4, 5
EPI_F16, EPI_F32, EPI_RESID_F32, EPI_SWIGLU = 0, 1, 2, 3
CLASSES = ("gemm", "attention", "norm_rope", "pool", "lm_head", "attention_tc", "lora")
