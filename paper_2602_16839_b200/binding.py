"""ctypes binding of libptenc.so: argument marshalling only.

Function names and argument order are those of include/ptenc.h.  Tensors are torch tensors used as device
memory; the binding passes `data_ptr()` and the current CUDA stream.  There is no fallback: if the library
is missing or fails to load, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libptenc.so")

PTENC_OK, PTENC_EINVAL, PTENC_ESHAPE, PTENC_EALIGN, PTENC_EWORKSPACE, PTENC_ECUDA, PTENC_EDEVICE_STATUS = (
    0, -1, -2, -3, -4, -5, -6)
PTENC_ELIMIT = -7
DTYPE_FP32, DTYPE_BF16 = 0, 1
NORM_ROW_L2, NORM_FROBENIUS, NORM_NONE = 0, 1, 2
POLICY_FIFO, POLICY_SCORE = 0, 1
(REGION_K, REGION_V, REGION_HEAD, REGION_COUNT, REGION_NAPP, REGION_NPINNED, REGION_STATE, REGION_TICKETS,
 REGION_STATUS) = range(9)

EXPORTS = ["ptenc_workspace_bytes", "ptenc_cache_create", "ptenc_cache_destroy", "ptenc_cache_reset",
           "ptenc_set_encoder", "ptenc_prefill", "ptenc_get_pinned", "ptenc_append_evict", "ptenc_decode_attn", "ptenc_encode", "ptenc_lora_apply", "ptenc_decode_step",
           "ptenc_host_staging_bytes", "ptenc_decode_step_host",
           "ptenc_get_ring", "ptenc_get_state", "ptenc_get_evicted", "ptenc_get_scores", "ptenc_cache_status", "ptenc_cache_info", "ptenc_attn_launch_info",
           "ptenc_workspace_region", "ptenc_time_next_attn", "ptenc_attn_rings_static", "ptenc_launch_count",
           "ptenc_strerror"]


class PtencConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "n_layers", "batch", "n_q_heads", "n_kv_heads", "head_dim", "window", "evict_chunk", "n_global",
        "rank", "dtype", "normalize_mode", "encode_enabled", "device", "attn_consumer_warps", "policy", "recent")]


class PtencError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python paper_2602_16839_b200/build.py` "
            "(there is no CPU or PyTorch fallback for this path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, u64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    cfgp = ctypes.POINTER(PtencConfig)
    lib.ptenc_workspace_bytes.argtypes = [cfgp, ctypes.POINTER(u64)]
    lib.ptenc_cache_create.argtypes = [cfgp, vp, u64, vp, ctypes.POINTER(vp)]
    lib.ptenc_cache_destroy.argtypes = [vp]
    lib.ptenc_cache_reset.argtypes = [vp, vp, vp]
    lib.ptenc_set_encoder.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.ptenc_prefill.argtypes = [vp, i32, vp, vp, vp, ctypes.c_int32, vp]
    lib.ptenc_get_pinned.argtypes = [vp, i32, vp, vp]
    lib.ptenc_append_evict.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.ptenc_decode_attn.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    lib.ptenc_encode.argtypes = [vp, i32, vp, vp, vp, ctypes.c_int32, vp]
    lib.ptenc_lora_apply.argtypes = [vp, i32, vp, vp, vp, vp, vp, ctypes.c_int32, ctypes.c_int32, vp]
    lib.ptenc_decode_step.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp]
    lib.ptenc_host_staging_bytes.argtypes = [vp, i32, ctypes.POINTER(u64)]
    lib.ptenc_decode_step_host.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, u64, vp]
    lib.ptenc_get_ring.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.ptenc_get_state.argtypes = [vp, i32, vp, vp]
    lib.ptenc_get_evicted.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.ptenc_get_scores.argtypes = [vp, i32, vp, vp, vp]
    lib.ptenc_cache_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32)]
    lib.ptenc_cache_info.argtypes = [vp] + [ctypes.POINTER(ctypes.c_int32)] * 3
    lib.ptenc_attn_launch_info.argtypes = [vp, i32] + [ctypes.POINTER(ctypes.c_int32)] * 3
    lib.ptenc_workspace_region.argtypes = [vp, i32, ctypes.POINTER(u64), ctypes.POINTER(u64)]
    lib.ptenc_time_next_attn.argtypes = [vp, vp, vp]
    lib.ptenc_attn_rings_static.argtypes = [cfgp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.ptenc_launch_count.argtypes = [vp, ctypes.POINTER(ctypes.c_int64)]
    lib.ptenc_strerror.argtypes = [i32]
    lib.ptenc_strerror.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name != "ptenc_strerror":
            getattr(lib, name).restype = ctypes.c_int
    return lib


lib = _load()


def strerror(code: int) -> str:
    return lib.ptenc_strerror(int(code)).decode()


def _check(rc: int, where: str) -> None:
    if rc != PTENC_OK:
        raise PtencError(rc, where)


def _ptr(t) -> int | None:
    if t is None:
        return None
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def make_config(*, n_layers, batch, n_q_heads, n_kv_heads, head_dim, window, evict_chunk=1, n_global=32,
                rank=32, dtype="bf16", normalize_mode=0, encode_enabled=1, device=0, attn_consumer_warps=0,
                policy=POLICY_FIFO, recent=0) -> PtencConfig:
    c = PtencConfig()
    c.n_layers, c.batch, c.n_q_heads, c.n_kv_heads, c.head_dim = n_layers, batch, n_q_heads, n_kv_heads, head_dim
    c.window, c.evict_chunk, c.n_global, c.rank = window, evict_chunk, n_global, rank
    c.dtype = {"fp32": DTYPE_FP32, "bf16": DTYPE_BF16}[dtype] if isinstance(dtype, str) else int(dtype)
    c.normalize_mode, c.encode_enabled, c.device = normalize_mode, encode_enabled, device
    c.attn_consumer_warps, c.policy, c.recent = attn_consumer_warps, policy, recent
    return c


def ptenc_workspace_bytes(cfg: PtencConfig) -> int:
    n = ctypes.c_size_t(0)
    _check(lib.ptenc_workspace_bytes(ctypes.byref(cfg), ctypes.byref(n)), "ptenc_workspace_bytes")
    return int(n.value)


def attn_rings_static(cfg: PtencConfig, K, V, head, count, q, out, active=None, lse_out=None, status_out=None):
    """ptenc_attn_rings_static: attention over caller-owned rings; the library allocates nothing (its scratch is a
    device array inside the library image).  All arguments are torch CUDA tensors (or None where optional)."""
    _check(lib.ptenc_attn_rings_static(ctypes.byref(cfg), _ptr(K), _ptr(V), _ptr(head), _ptr(count), _ptr(q),
                                       _ptr(active), _ptr(out), _ptr(lse_out), _ptr(status_out), _stream()),
           "ptenc_attn_rings_static")


class Cache:
    """Owns the torch-allocated workspace and the library handle.  Methods mirror the C entry points."""

    def __init__(self, cfg: PtencConfig):
        if not torch.cuda.is_available():
            raise RuntimeError("ptenc needs a CUDA device; there is no CPU path")
        self.cfg = cfg
        self.device = torch.device("cuda", cfg.device)
        self.torch_dtype = torch.float32 if cfg.dtype == DTYPE_FP32 else torch.bfloat16
        nbytes = ptenc_workspace_bytes(cfg)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 1023) // 1024 * 1024
            h = ctypes.c_void_p()
            _check(lib.ptenc_cache_create(ctypes.byref(cfg), self._ws_ptr, nbytes, _stream(), ctypes.byref(h)),
                   "ptenc_cache_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib.ptenc_cache_destroy(self._h)
            self._h = None
            self.workspace = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- entry points --------------------------------------------------------------------------------
    def reset(self, seq_mask=None):
        _check(lib.ptenc_cache_reset(self._h, _ptr(seq_mask), _stream()), "ptenc_cache_reset")

    def set_encoder(self, layer, Wq_a, Wk_a, Wv_a, q_g, k_g=None, v_g=None):
        _check(lib.ptenc_set_encoder(self._h, layer, _ptr(Wq_a), _ptr(Wk_a), _ptr(Wv_a), _ptr(q_g), _ptr(k_g),
                                     _ptr(v_g), _stream()), "ptenc_set_encoder")

    def prefill(self, layer, K_p, V_p, n_prompt, p_max):
        _check(lib.ptenc_prefill(self._h, layer, _ptr(K_p), _ptr(V_p), _ptr(n_prompt), int(p_max), _stream()),
               "ptenc_prefill")

    def get_pinned(self, layer):
        n = torch.empty(self.cfg.batch, dtype=torch.int32, device=self.device)
        _check(lib.ptenc_get_pinned(self._h, layer, _ptr(n), _stream()), "ptenc_get_pinned")
        return n

    def append_evict(self, layer, k_new, v_new, active=None, slot_out=None, evict_first_out=None,
                     n_evicted_out=None):
        _check(lib.ptenc_append_evict(self._h, layer, _ptr(k_new), _ptr(v_new), _ptr(active), _ptr(slot_out),
                                      _ptr(evict_first_out), _ptr(n_evicted_out), _stream()), "ptenc_append_evict")

    def decode_attn(self, layer, q, out, active=None, lse_out=None):
        _check(lib.ptenc_decode_attn(self._h, layer, _ptr(q), _ptr(active), _ptr(out), _ptr(lse_out), _stream()),
               "ptenc_decode_attn")

    def encode(self, layer, K_e=None, V_e=None, n_evicted=None, m_max=0):
        _check(lib.ptenc_encode(self._h, layer, _ptr(K_e), _ptr(V_e), _ptr(n_evicted), int(m_max), _stream()),
               "ptenc_encode")

    def lora_apply(self, layer, A, Bm, x, y, active=None):
        """y += A (S (Bm x)) per sequence; A [.., d_out, G], Bm [.., r, d_in], x [.., B, d_in], y [.., B, d_out]."""
        _check(lib.ptenc_lora_apply(self._h, layer, _ptr(A), _ptr(Bm), _ptr(x), _ptr(y), _ptr(active),
                                    int(x.shape[-1]), int(y.shape[-1]), _stream()), "ptenc_lora_apply")

    def decode_step(self, layer, q, k_new, v_new, out, active=None):
        _check(lib.ptenc_decode_step(self._h, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(active), _ptr(out),
                                     _stream()), "ptenc_decode_step")

    def host_staging_bytes(self, layer) -> int:
        n = ctypes.c_size_t(0)
        _check(lib.ptenc_host_staging_bytes(self._h, layer, ctypes.byref(n)), "ptenc_host_staging_bytes")
        return int(n.value)

    def decode_step_host(self, layer, q_host, k_host, v_host, out_host, dev_staging, active_host=None):
        """Host tensors in (pinned), host tensor out; `dev_staging` is a device uint8 tensor."""
        _check(lib.ptenc_decode_step_host(self._h, layer, _ptr(q_host), _ptr(k_host), _ptr(v_host),
                                          _ptr(active_host), _ptr(out_host), _ptr(dev_staging),
                                          dev_staging.numel(), _stream()), "ptenc_decode_step_host")

    def get_ring(self, layer):
        B = self.cfg.batch
        head = torch.empty(B, dtype=torch.int32, device=self.device)
        count = torch.empty(B, dtype=torch.int32, device=self.device)
        n_app = torch.empty(B, dtype=torch.int64, device=self.device)
        _check(lib.ptenc_get_ring(self._h, layer, _ptr(head), _ptr(count), _ptr(n_app), _stream()), "ptenc_get_ring")
        return head, count, n_app

    def get_state(self, layer):
        S = torch.empty(self.cfg.batch, self.cfg.n_global, self.cfg.rank, dtype=torch.float32, device=self.device)
        _check(lib.ptenc_get_state(self._h, layer, _ptr(S), _stream()), "ptenc_get_state")
        return S

    def get_evicted(self, layer):
        """(tokens [B, E] int64 oldest first, slots [B, E] int32, n_evicted [B] int32) of the last append (score policy)."""
        B, E = self.cfg.batch, self.cfg.evict_chunk
        tok = torch.full((B, E), -1, dtype=torch.int64, device=self.device)
        slot = torch.full((B, E), -1, dtype=torch.int32, device=self.device)
        n = torch.zeros(B, dtype=torch.int32, device=self.device)
        _check(lib.ptenc_get_evicted(self._h, layer, _ptr(tok), _ptr(slot), _ptr(n), _stream()), "ptenc_get_evicted")
        return tok, slot, n

    def get_scores(self, layer):
        """(score [B, W] fp32, token [B, W] int32, -1 where the slot holds no unpinned token) (score policy)."""
        B, W = self.cfg.batch, self.cfg.window
        score = torch.empty(B, W, dtype=torch.float32, device=self.device)
        token = torch.empty(B, W, dtype=torch.int32, device=self.device)
        _check(lib.ptenc_get_scores(self._h, layer, _ptr(score), _ptr(token), _stream()), "ptenc_get_scores")
        return score, token

    def status(self) -> int:
        st = ctypes.c_int32(0)
        rc = lib.ptenc_cache_status(self._h, ctypes.byref(st))
        if rc not in (PTENC_OK, PTENC_EDEVICE_STATUS):
            raise PtencError(rc, "ptenc_cache_status")
        return int(st.value)

    def info(self) -> dict:
        a, b, e = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_int32(0)
        _check(lib.ptenc_cache_info(self._h, ctypes.byref(a), ctypes.byref(b), ctypes.byref(e)), "ptenc_cache_info")
        return {"tensor_core_attn": bool(a.value), "attn_grid": int(b.value), "tensor_core_encode": bool(e.value)}

    def attn_launch_info(self, layer=-1) -> dict:
        w, t, s = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_int32(0)
        _check(lib.ptenc_attn_launch_info(self._h, layer, ctypes.byref(w), ctypes.byref(t), ctypes.byref(s)),
               "ptenc_attn_launch_info")
        return {"consumer_warps": int(w.value), "tile_tokens": int(t.value), "stages": int(s.value)}

    def workspace_region(self, region: int):
        """(device pointer, bytes) of one part of the decode state inside the workspace."""
        off, n = ctypes.c_size_t(0), ctypes.c_size_t(0)
        _check(lib.ptenc_workspace_region(self._h, int(region), ctypes.byref(off), ctypes.byref(n)),
               "ptenc_workspace_region")
        return self._ws_ptr + int(off.value), int(n.value)

    def time_next_attn(self, ev_begin, ev_end):
        """ev_begin/ev_end: torch.cuda.Event(enable_timing=True) that have been recorded once (so that their
        CUDA handles exist); they are re-recorded around the next attention kernel."""
        _check(lib.ptenc_time_next_attn(self._h, ev_begin.cuda_event, ev_end.cuda_event), "ptenc_time_next_attn")

    def launch_count(self) -> int:
        n = ctypes.c_int64(0)
        _check(lib.ptenc_launch_count(self._h, ctypes.byref(n)), "ptenc_launch_count")
        return int(n.value)
