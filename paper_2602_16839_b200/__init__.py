"""B200-native decode hot path of Progressive Thought Encoding (ring KV cache, GQA decode attention,
progressive encoding of evicted tokens).  The compute lives in libptenc.so (CUDA, sm_100a); this package is
the thin binding over its C ABI."""
from .binding import (Cache, attn_rings_static, PtencConfig, PtencError, lib, make_config, ptenc_workspace_bytes, strerror,  # noqa: F401
                      EXPORTS, LIB_PATH)
