"""Thin ctypes binding over libpt.so (see include/pt.h for the contract of every call).

Only argument marshalling lives here; every step of the forward pass runs in the library's
CUDA kernels.  PyTorch is used for device memory and streams: the ``Model`` helper owns the
torch tensors that back the packed weights, the KV pool and the workspace, and hands their
raw pointers to the C ABI.  Without the compiled library every call raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpt.so")

PT_OK = 0
STATUS = {0: "PT_OK", 1: "PT_ERR_INVALID_ARG", 2: "PT_ERR_BAD_CONFIG", 3: "PT_ERR_UNSUPPORTED",
          4: "PT_ERR_BUFFER_TOO_SMALL", 5: "PT_ERR_CACHE_FULL", 6: "PT_ERR_MISALIGNED", 7: "PT_ERR_CUDA",
          8: "PT_ERR_DEVICE_BOUNDS", 9: "PT_ERR_DEVICE_TIMEOUT", 10: "PT_ERR_STATE"}
PT_F32, PT_BF16 = 0, 1
PT_KV_MODEL, PT_KV_E4M3 = 0, 1
KIND = {"wq": 0, "wk": 1, "wv": 2, "wo": 3, "wg": 4, "wu": 5, "wd": 6, "g1": 7, "g2": 8, "wr": 9}


class PtError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"{STATUS.get(code, code)}: {msg}")
        self.code = code


class pt_config(C.Structure):
    _fields_ = [("T", C.c_int32), ("D", C.c_int32), ("L", C.c_int32), ("hidden", C.c_int32),
                ("heads", C.c_int32), ("kv_heads", C.c_int32), ("ffn", C.c_int32),
                ("rope_base", C.c_float), ("rms_eps", C.c_float), ("dtype", C.c_int32),
                ("sync_op", C.c_int32), ("max_pos", C.c_int32), ("flags", C.c_int32),
                ("experts", C.c_int32), ("top_k", C.c_int32)]


_P, _I32, _I64, _SZ = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
_PROTOS = {
    "pt_model_create": (_I32, [C.POINTER(pt_config), C.POINTER(_P)]),
    "pt_model_destroy": (None, [_P]),
    "pt_model_weight_bytes": (_I32, [_P, C.POINTER(_SZ)]),
    "pt_model_bind_weights": (_I32, [_P, _P, _SZ]),
    "pt_model_set_weight": (_I32, [_P, _I32, _I32, _I32, _P, _P]),
    "pt_model_set_expert_weight": (_I32, [_P, _I32, _I32, _I32, _I32, _P, _P]),
    "pt_sync_count": (_I32, [_P]),
    "pt_model_set_track_group": (_I32, [_P, _I32, _P, _P]),
    "pt_kv_cache_bytes": (_I32, [_P, _I32, _I32, C.POINTER(_SZ)]),
    "pt_kv_cache_alloc": (_I32, [_P, _I32, _I32, _P, _SZ, C.POINTER(_P)]),
    "pt_kv_cache_bytes_ex": (_I32, [_P, _I32, _I32, _I32, C.POINTER(_SZ)]),
    "pt_kv_cache_alloc_ex": (_I32, [_P, _I32, _I32, _I32, _P, _SZ, C.POINTER(_P)]),
    "pt_kv_scale_slot": (_I32, [_P, _I32, _I32, _I32, _I32, _I32, _I32, C.POINTER(_I64)]),
    "pt_workspace_bytes_ex": (_I32, [_P, _I64, _I32, _I32, _I32, _I64, C.POINTER(_SZ)]),
    "pt_kernel_kv_quant_e4m3": (_I32, [_P, _P, _P, _I64, _P, _P]),
    "pt_kv_cache_free": (None, [_P]),
    "pt_kv_set_free_list": (_I32, [_P, C.POINTER(_I32), _I32]),
    "pt_kv_seq_reserve": (_I32, [_P, _I32, _I32]),
    "pt_kv_seq_release": (_I32, [_P, _I32]),
    "pt_kv_seq_len": (_I32, [_P, _I32, C.POINTER(_I32)]),
    "pt_kv_seq_truncate": (_I32, [_P, _I32, _I32]),
    "pt_kv_block_table": (_I32, [_P, _I32, C.POINTER(_I32), _I32, C.POINTER(_I32)]),
    "pt_kv_slot": (_I32, [_P, _I32, _I32, _I32, _I32, _I32, _I32, C.POINTER(_I64)]),
    "pt_workspace_bytes": (_I32, [_P, _I64, _I32, _I32, C.POINTER(_SZ)]),
    "pt_prefill": (_I32, [_P, _P, _P, _I64, _I32, _I32, C.POINTER(_I32), _P, _P, _SZ, _P]),
    "pt_decode_step": (_I32, [_P, _P, _P, _I64, _I32, C.POINTER(_I32), _P, _P, _SZ, _P]),
    "pt_lm_bytes": (_I32, [_P, _I32, C.POINTER(_SZ)]),
    "pt_lm_bind": (_I32, [_P, _I32, _P, _SZ]),
    "pt_lm_set": (_I32, [_P, _I32, _P, _P]),
    "pt_embed": (_I32, [_P, _P, _I64, _P, _P]),
    "pt_lm_workspace_bytes": (_I32, [_P, _I64, C.POINTER(_SZ)]),
    "pt_lm_head": (_I32, [_P, _P, _I64, _I64, _P, _P, _P, _SZ, _P]),
    "pt_generate_workspace_bytes": (_I32, [_P, _I32, _I32, _I32, C.POINTER(_SZ)]),
    "pt_generate": (_I32, [_P, _P, _P, _I32, _I32, _I32, C.POINTER(_I32), _P, _P, _P, _SZ, _P]),
    "pt_set_debug_tap": (_I32, [_P, _I32, _P]),
    "pt_device_status": (_I32, [_P, _P, C.POINTER(_I32), C.POINTER(_I32)]),
    "pt_profile_enable": (_I32, [_P, _I32]),
    "pt_profile_read": (_I32, [_P, C.POINTER(C.c_float), C.POINTER(_I64)]),
    "pt_launch_count": (_I64, []),
    "pt_kernel_gemm_bf16": (_I32, [_P, _P, _P, _I32, _I32, _I32, _I32, _I32, _I32, _P, _P]),
    "pt_kernel_prefill_attn": (_I32, [_P, _P, _I64, _P, _I32, _P, _I32, _I32, _I32, _I32, _I32, _I32, _I32, _I32, _P, _I32, _P, _P]),
    "pt_kernel_decode_attn_scratch_bytes": (_I32, [_I32, _I32, _I32, _I32, C.POINTER(_SZ)]),
    "pt_kernel_decode_attn": (_I32, [_P, _P, _I64, _P, _I32, C.POINTER(_I32), _I32, _I32, _I32, _I32, _I32, _I32, _I32,
                                     _P, _P, _SZ, _P, _P]),
    "pt_kernel_decode_attn_static": (_I32, [_P, _P, _I64, _P, _I32, C.POINTER(_I32), _I32, _I32, _I32, _I32, _I32, _I32, _I32,
                                            _P, _P, _P]),
    "pt_kernel_decode_attn_e4m3": (_I32, [_P, _P, _I64, _P, _I64, _P, _I32, C.POINTER(_I32), _I32, _I32, _I32, _I32, _I32, _I32,
                                          _P, _I32, _P, _SZ, _P, _P]),
    "pt_kernel_wait_selftest": (_I32, [_P, C.c_uint64, _P]),
    "pt_last_error": (C.c_char_p, []),
}
EXPORTS = tuple(_PROTOS)
_lib = None


def lib() -> C.CDLL:
    """Load libpt.so once; raise if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2602_07306_b200.build` "
                               "(there is no CPU fallback)")
        l = C.CDLL(LIB_PATH)
        for name, (res, args) in _PROTOS.items():
            f = getattr(l, name)
            f.restype, f.argtypes = res, args
        _lib = l
    return _lib


def check(code: int) -> None:
    if code != PT_OK:
        raise PtError(code, lib().pt_last_error().decode())


def _i32arr(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(C.POINTER(_I32))


class Model:
    """A PT model with its packed weights on one CUDA device (torch owns the memory)."""

    def __init__(self, *, T, D, L, hidden, heads, kv_heads, ffn, dtype="bf16", rope_base=10000.0,
                 rms_eps=1e-6, sync_op="sum", max_pos=4096, simt=False, flags=0, experts=0, top_k=0, device="cuda:0"):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        self.cfg = pt_config(T, D, L, hidden, heads, kv_heads, ffn, rope_base, rms_eps,
                             PT_BF16 if dtype == "bf16" else PT_F32, 1 if sync_op == "mean" else 0,
                             max_pos, (1 if simt else 0) | int(flags), experts, top_k)
        self.dtype = dtype
        self.tdtype = torch.bfloat16 if dtype == "bf16" else torch.float32
        self.h = _P()
        check(lib().pt_model_create(C.byref(self.cfg), C.byref(self.h)))
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: there is no CPU path")
        n = _SZ()
        check(lib().pt_model_weight_bytes(self.h, C.byref(n)))
        self.weight_bytes = n.value
        with torch.cuda.device(self.device):
            self.wbuf = torch.empty(n.value, dtype=torch.uint8, device=self.device)
            check(lib().pt_model_bind_weights(self.h, self.wbuf.data_ptr(), n.value))
        self.ws = None
        self.ws_key = (0, 0, 0)
        self._tap = None

    def close(self):
        if self.h:
            lib().pt_model_destroy(self.h)
            self.h = _P()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _stream(self):
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def set_weight(self, t: int, l: int, kind: str, w) -> None:
        """w: numpy float32 array or torch tensor, [out, in] (gains: [hidden])."""
        torch = self.torch
        if isinstance(w, np.ndarray):
            w = torch.from_numpy(np.ascontiguousarray(w))
        want = torch.float32 if kind in ("g1", "g2", "wr") else self.tdtype
        w = w.to(device=self.device, dtype=want).contiguous()
        with torch.cuda.device(self.device):
            if self.cfg.experts and kind in ("wg", "wu", "wd"):       # PT-MoE: [experts, ...], one call per expert
                for e in range(self.cfg.experts):
                    check(lib().pt_model_set_expert_weight(self.h, t, l, e, KIND[kind], w[e].data_ptr(), self._stream()))
            else:
                check(lib().pt_model_set_weight(self.h, t, l, KIND[kind], w.data_ptr(), self._stream()))
            torch.cuda.current_stream().synchronize()      # w may be freed after return

    def load(self, source) -> None:
        """source.get(t, l) -> dict kind -> float32 numpy array."""
        for l in range(self.cfg.L):
            for t in range(self.cfg.T):
                for k, w in source.get(t, l).items():
                    self.set_weight(t, l, k, w)

    def init_random(self, seed: int = 0, std: float = 0.02) -> None:
        """Weights N(0, std), gains 1, drawn on the device (for timing runs)."""
        torch = self.torch
        c = self.cfg
        dh = c.hidden // c.heads
        g = torch.Generator(device=self.device).manual_seed(seed)
        shapes = {"wq": (c.heads * dh, c.hidden), "wk": (c.kv_heads * dh, c.hidden), "wv": (c.kv_heads * dh, c.hidden),
                  "wo": (c.hidden, c.heads * dh), "wg": (c.ffn, c.hidden), "wu": (c.ffn, c.hidden), "wd": (c.hidden, c.ffn)}
        ones = torch.ones(c.hidden, dtype=torch.float32, device=self.device)
        with torch.cuda.device(self.device):
            for l in range(c.L):
                for t in range(c.T):
                    for k, shp in shapes.items():
                        for e in range(c.experts if c.experts and k in ("wg", "wu", "wd") else 1):
                            w = (torch.randn(shp, generator=g, device=self.device, dtype=torch.float32) * std).to(self.tdtype)
                            if c.experts and k in ("wg", "wu", "wd"):
                                check(lib().pt_model_set_expert_weight(self.h, t, l, e, KIND[k], w.data_ptr(), self._stream()))
                            else:
                                check(lib().pt_model_set_weight(self.h, t, l, KIND[k], w.data_ptr(), self._stream()))
                    if c.experts:
                        wr = torch.randn((c.experts, c.hidden), generator=g, device=self.device, dtype=torch.float32) * std
                        check(lib().pt_model_set_weight(self.h, t, l, KIND["wr"], wr.data_ptr(), self._stream()))
                    for k in ("g1", "g2"):
                        check(lib().pt_model_set_weight(self.h, t, l, KIND[k], ones.data_ptr(), self._stream()))
            torch.cuda.synchronize()

    def set_track_group(self, world_tracks: int, allreduce) -> None:
        """This model holds cfg.T of `world_tracks` tracks; `allreduce(t)` must sum the fp32 CUDA tensor t in
        place over all ranks on the current stream (e.g. torch.distributed.all_reduce).  None clears it."""
        if allreduce is None:
            check(lib().pt_model_set_track_group(self.h, 0, None, None))
            self._ar_cb = None
            return
        torch = self.torch

        def hook(user, ptr, count, stream):
            try:
                off = ptr - self.ws.data_ptr()
                assert 0 <= off and off + 4 * count <= self.ws.numel(), "buffer outside the workspace"
                allreduce(self.ws[off:off + 4 * count].view(torch.float32))
                return 0
            except Exception as e:      # never let an exception cross the C boundary
                self._ar_error = e
                return 1
        self._ar_cb = C.CFUNCTYPE(_I32, _P, _P, _I64, _P)(hook)
        check(lib().pt_model_set_track_group(self.h, world_tracks, C.cast(self._ar_cb, _P), None))

    def sync_count(self) -> int:
        return lib().pt_sync_count(self.h)

    def new_cache(self, num_pages: int, page_size: int = 16, free_order=None, kv_dtype: str = "model") -> "Cache":
        """kv_dtype "model" keeps K and V in the model dtype, "e4m3" stores 8-bit codes and one scale per vector."""
        return Cache(self, num_pages, page_size, free_order, kv_dtype=kv_dtype)

    def workspace(self, tokens: int, batch: int, page_size: int, kv_dtype: int = PT_KV_MODEL, context: int = 0):
        """Workspace for calls of up to `tokens` tokens / `batch` sequences; with an E4M3 cache `context` bounds the
        keys a prefill call attends to (sum over its sequences of the length after the call, each rounded up to 16)."""
        key = self.ws_key + (0, 0) if len(self.ws_key) == 3 else self.ws_key
        if (self.ws is None or tokens > key[0] or batch > key[1] or page_size < key[2] or kv_dtype > key[3] or context > key[4]):
            tokens, batch, context = max(tokens, key[0]), max(batch, key[1]), max(context, key[4])
            kv_dtype = max(kv_dtype, key[3])
            page_size = min(page_size, key[2]) if key[2] else page_size
            n = _SZ()
            check(lib().pt_workspace_bytes_ex(self.h, tokens, batch, page_size, kv_dtype, context, C.byref(n)))
            self.ws = None
            self.ws = self.torch.empty(n.value, dtype=self.torch.uint8, device=self.device)
            self.ws_key = (tokens, batch, page_size, kv_dtype, context)
        return self.ws

    def set_tap(self, layer: int | None, tokens: int = 0):
        """layer None: off; -1: all layers.  Returns the tap tensor [nl, 2, T, tokens, hidden]."""
        torch = self.torch
        if layer is None:
            check(lib().pt_set_debug_tap(self.h, 0, None))
            self._tap = None
            return None
        nl = self.cfg.L if layer == -1 else 1
        self._tap = torch.zeros((nl, 2, self.cfg.T, tokens, self.cfg.hidden), dtype=torch.float32, device=self.device)
        check(lib().pt_set_debug_tap(self.h, layer, self._tap.data_ptr()))
        return self._tap

    def prefill(self, cache: "Cache", x, seq_ids, out=None):
        """x: torch tensor [T, B, S, H] (or [1, B, S, H] = shared input) in the model dtype."""
        torch = self.torch
        assert x.is_cuda and x.dtype == self.tdtype and x.is_contiguous()
        Tn, B, S, H = x.shape
        stride = 0 if Tn == 1 and self.cfg.T > 1 else B * S * H
        if out is None:
            out = torch.empty((B, S, H), dtype=torch.float32, device=self.device)
        ids, pids = _i32arr(seq_ids)
        assert len(ids) == B
        ctx = 0
        if cache.kv_dtype == PT_KV_E4M3:
            ctx = sum((cache.length(int(s)) + S + 15) // 16 * 16 for s in ids)
        ws = self.workspace(B * S, B, cache.page_size, cache.kv_dtype, ctx)
        with torch.cuda.device(self.device):
            check(lib().pt_prefill(self.h, cache.h, x.data_ptr(), stride, B, S, pids, out.data_ptr(),
                                   ws.data_ptr(), ws.numel(), self._stream()))
        return out

    def decode_step(self, cache: "Cache", x, seq_ids, out=None):
        """x: torch tensor [T, B, H] (or [1, B, H]) in the model dtype -> fp32 [B, H]."""
        torch = self.torch
        assert x.is_cuda and x.dtype == self.tdtype and x.is_contiguous()
        Tn, B, H = x.shape
        stride = 0 if Tn == 1 and self.cfg.T > 1 else B * H
        if out is None:
            out = torch.empty((B, H), dtype=torch.float32, device=self.device)
        ws = self.workspace(B, B, cache.page_size, cache.kv_dtype, 0)
        ids, pids = _i32arr(seq_ids)
        assert len(ids) == B
        with torch.cuda.device(self.device):
            check(lib().pt_decode_step(self.h, cache.h, x.data_ptr(), stride, B, pids, out.data_ptr(),
                                       ws.data_ptr(), ws.numel(), self._stream()))
        return out

    # ---- ends of the model -------------------------------------------------------------------
    def load_lm(self, table, head, gain) -> None:
        """table, head: [vocab, hidden]; gain: [hidden] (numpy or torch); stored in the model dtype / fp32."""
        torch = self.torch
        as_t = lambda a: torch.from_numpy(np.ascontiguousarray(a)) if isinstance(a, np.ndarray) else a
        table, head, gain = as_t(table), as_t(head), as_t(gain)
        self.vocab = table.shape[0]
        n = _SZ()
        check(lib().pt_lm_bytes(self.h, self.vocab, C.byref(n)))
        with torch.cuda.device(self.device):
            self.lm_buf = torch.empty(n.value, dtype=torch.uint8, device=self.device)
            check(lib().pt_lm_bind(self.h, self.vocab, self.lm_buf.data_ptr(), n.value))
            for kind, w, dt in ((0, table, self.tdtype), (1, head, self.tdtype), (2, gain, torch.float32)):
                w = w.to(device=self.device, dtype=dt).contiguous()
                check(lib().pt_lm_set(self.h, kind, w.data_ptr(), self._stream()))
                torch.cuda.current_stream().synchronize()

    def embed(self, tokens):
        """tokens: int32 CUDA tensor of any shape -> [..., hidden] in the model dtype."""
        torch = self.torch
        assert tokens.is_cuda and tokens.dtype == torch.int32 and tokens.is_contiguous()
        x = torch.empty(tuple(tokens.shape) + (self.cfg.hidden,), dtype=self.tdtype, device=self.device)
        with torch.cuda.device(self.device):
            check(lib().pt_embed(self.h, tokens.data_ptr(), tokens.numel(), x.data_ptr(), self._stream()))
        return x

    def lm_head(self, h, want_tokens=True):
        """h: fp32 CUDA [n, hidden] (contiguous) -> (logits fp32 [n, vocab], greedy tokens int32 [n] or None)."""
        torch = self.torch
        assert h.is_cuda and h.dtype == torch.float32 and h.is_contiguous() and h.dim() == 2
        n = h.shape[0]
        logits = torch.empty((n, self.vocab), dtype=torch.float32, device=self.device)
        tok = torch.empty(n, dtype=torch.int32, device=self.device) if want_tokens else None
        nb = _SZ()
        check(lib().pt_lm_workspace_bytes(self.h, n, C.byref(nb)))
        ws = torch.empty(nb.value, dtype=torch.uint8, device=self.device)
        with torch.cuda.device(self.device):
            check(lib().pt_lm_head(self.h, h.data_ptr(), h.shape[1], n, logits.data_ptr(), tok.data_ptr() if want_tokens else None,
                                   ws.data_ptr(), ws.numel(), self._stream()))
        return logits, tok

    def generate(self, cache: "Cache", prompt, n_new: int, seq_ids, want_logits=False):
        """prompt: int32 CUDA [B, S] -> (tokens int32 [B, n_new], logits fp32 [B, n_new, vocab] or None)."""
        torch = self.torch
        assert prompt.is_cuda and prompt.dtype == torch.int32 and prompt.is_contiguous()
        B, S = prompt.shape
        out = torch.empty((B, n_new), dtype=torch.int32, device=self.device)
        logits = torch.empty((B, n_new, self.vocab), dtype=torch.float32, device=self.device) if want_logits else None
        nb = _SZ()
        check(lib().pt_generate_workspace_bytes(self.h, B, S, cache.page_size, C.byref(nb)))
        if getattr(self, "gen_ws", None) is None or self.gen_ws.numel() < nb.value:
            self.gen_ws = None
            self.gen_ws = torch.empty(nb.value, dtype=torch.uint8, device=self.device)
        ids, pids = _i32arr(seq_ids)
        with torch.cuda.device(self.device):
            check(lib().pt_generate(self.h, cache.h, prompt.data_ptr(), B, S, n_new, pids, out.data_ptr(),
                                    logits.data_ptr() if want_logits else None, self.gen_ws.data_ptr(), self.gen_ws.numel(), self._stream()))
        return out, logits

    PROF_NAMES = ("attention", "gemm_qkv", "gemm_out", "gemm_gate_up", "gemm_down", "gemm_down_sync", "other")

    def profile(self, on, only=None) -> None:
        """on False / True: no launch / every launch bracketed with events; only=("attention", ...) brackets
        the launches of those categories alone."""
        code = int(bool(on))
        if on and only:
            code = sum(2 << self.PROF_NAMES.index(n) for n in only)
        check(lib().pt_profile_enable(self.h, code))

    def profile_read(self) -> dict:
        """Device milliseconds and launches per kernel category since the last read."""
        ms = (C.c_float * 7)()
        n = (_I64 * 7)()
        with self.torch.cuda.device(self.device):
            check(lib().pt_profile_read(self.h, ms, n))
        return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(self.PROF_NAMES)}

    def device_status(self) -> tuple[int, int]:
        code, detail = _I32(), _I32()
        with self.torch.cuda.device(self.device):
            check(lib().pt_device_status(self.h, self._stream(), C.byref(code), C.byref(detail)))
        return code.value, detail.value


class Cache:
    """Paged KV cache: torch owns the pool, the library's host allocator owns the page tables."""

    def __init__(self, model: Model, num_pages: int, page_size: int = 16, free_order=None, fill=None, kv_dtype: str = "model"):
        torch = model.torch
        self.model, self.num_pages, self.page_size = model, num_pages, page_size
        self.kv_dtype = {"model": PT_KV_MODEL, "e4m3": PT_KV_E4M3}[kv_dtype]
        n = _SZ()
        check(lib().pt_kv_cache_bytes_ex(model.h, num_pages, page_size, self.kv_dtype, C.byref(n)))
        self.bytes = n.value
        if self.kv_dtype == PT_KV_E4M3:
            # one byte buffer: the codes, then the fp32 scales (views below)
            self.pool = torch.empty(n.value, dtype=torch.uint8, device=model.device)
            c = model.cfg
            vecs = c.T * c.L * num_pages * 2 * c.kv_heads * page_size
            dh = c.hidden // c.heads
            self.codes = self.pool[: vecs * dh]
            self.scales = self.pool[n.value - vecs * 4:].view(torch.float32)
        else:
            self.pool = torch.empty(n.value // (2 if model.dtype == "bf16" else 4), dtype=model.tdtype, device=model.device)
        self.h = _P()
        check(lib().pt_kv_cache_alloc_ex(model.h, num_pages, page_size, self.kv_dtype, self.pool.data_ptr(), n.value, C.byref(self.h)))
        if free_order is not None:
            a, p = _i32arr(free_order)
            check(lib().pt_kv_set_free_list(self.h, p, len(a)))

    def close(self):
        if self.h:
            lib().pt_kv_cache_free(self.h)
            self.h = _P()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reserve(self, seq: int, new_len: int):
        check(lib().pt_kv_seq_reserve(self.h, seq, new_len))

    def release(self, seq: int):
        check(lib().pt_kv_seq_release(self.h, seq))

    def truncate(self, seq: int, n: int):
        check(lib().pt_kv_seq_truncate(self.h, seq, n))

    def length(self, seq: int) -> int:
        v = _I32()
        check(lib().pt_kv_seq_len(self.h, seq, C.byref(v)))
        return v.value

    def block_table(self, seq: int) -> list[int]:
        n = _I32()
        check(lib().pt_kv_block_table(self.h, seq, None, 0, C.byref(n)))
        buf = (_I32 * max(1, n.value))()
        check(lib().pt_kv_block_table(self.h, seq, buf, n.value, C.byref(n)))
        return list(buf[: n.value])

    def slot(self, t: int, l: int, seq: int, pos: int, kv: int, head: int) -> int:
        v = _I64()
        check(lib().pt_kv_slot(self.h, t, l, seq, pos, kv, head, C.byref(v)))
        return v.value

    def scale_slot(self, t: int, l: int, seq: int, pos: int, kv: int, head: int) -> int:
        """E4M3 caches: byte offset inside the pool of the fp32 scale of the vector `slot` addresses."""
        v = _I64()
        check(lib().pt_kv_scale_slot(self.h, t, l, seq, pos, kv, head, C.byref(v)))
        return v.value

    def dequantized(self):
        """E4M3 caches: code * scale of the whole pool as a float32 CUDA tensor [T, L, pages, 2, kv_heads, page, dh]."""
        torch = self.model.torch
        c = self.model.cfg
        dh = c.hidden // c.heads
        shape = (c.T, c.L, self.num_pages, 2, c.kv_heads, self.page_size)
        codes = self.codes.view(torch.float8_e4m3fn).to(torch.float32).view(shape + (dh,))
        return codes * self.scales.view(shape + (1,))


def kernel_gemm_bf16(a, w, bn: int = 0, fold_tracks: bool = False):
    """a [T, M, K], w [T, N, K] bf16 CUDA tensors -> fp32 [T, M, N] ([1, M, N] when folding tracks)."""
    import torch
    T, M, K = a.shape
    N = w.shape[1]
    assert a.is_contiguous() and w.is_contiguous() and a.dtype == w.dtype == torch.bfloat16
    c = torch.empty((1 if fold_tracks else T, M, N), dtype=torch.float32, device=a.device)
    status = torch.zeros(16, dtype=torch.int32, device=a.device)
    with torch.cuda.device(a.device):
        check(lib().pt_kernel_gemm_bf16(a.data_ptr(), w.data_ptr(), c.data_ptr(), T, M, N, K, bn, int(fold_tracks),
                                        status.data_ptr(), torch.cuda.current_stream().cuda_stream))
    return c, status


def kernel_kv_quant_e4m3(src):
    """src: bf16 CUDA tensor [n, 128] -> (codes uint8 [n, 128], scales fp32 [n], status int32[16])."""
    import torch
    assert src.is_cuda and src.dtype == torch.bfloat16 and src.is_contiguous() and src.shape[1] == 128
    n = src.shape[0]
    codes = torch.empty((n, 128), dtype=torch.uint8, device=src.device)
    scales = torch.empty(n, dtype=torch.float32, device=src.device)
    status = torch.zeros(16, dtype=torch.int32, device=src.device)
    with torch.cuda.device(src.device):
        check(lib().pt_kernel_kv_quant_e4m3(src.data_ptr(), codes.data_ptr(), scales.data_ptr(), n, status.data_ptr(),
                                            torch.cuda.current_stream().cuda_stream))
    return codes, scales, status


def kernel_wait_selftest(limit_ns: int, device="cuda:0"):
    """Run the library's bounded wait on a barrier nothing arrives at; returns the status block (int32[16], CUDA)."""
    import torch
    status = torch.zeros(16, dtype=torch.int32, device=device)
    with torch.cuda.device(status.device):
        check(lib().pt_kernel_wait_selftest(status.data_ptr(), int(limit_ns), torch.cuda.current_stream().cuda_stream))
    return status


def kernel_decode_attn(q, pool_l, block_table, kv_len, *, nq, nkv, dh, ps, scratch=None):
    """q bf16 [T, B, nq*dh]; pool_l bf16 [T, pages, 2, nkv, ps, dh]; block_table int32 [B, maxp] (CUDA);
    kv_len: host ints [B].  Returns (out bf16 [T, B, nq*dh], status int32[16])."""
    import torch
    T, B, _ = q.shape
    pages = pool_l.shape[1]
    assert q.is_contiguous() and pool_l.is_contiguous() and block_table.is_contiguous()
    assert q.dtype == pool_l.dtype == torch.bfloat16 and block_table.dtype == torch.int32
    out = torch.empty_like(q)
    status = torch.zeros(16, dtype=torch.int32, device=q.device)
    n = _SZ()
    check(lib().pt_kernel_decode_attn_scratch_bytes(T, B, nq, dh, C.byref(n)))
    if scratch is None:
        scratch = torch.empty(n.value, dtype=torch.uint8, device=q.device)
    lens, plens = _i32arr(kv_len)
    with torch.cuda.device(q.device):
        check(lib().pt_kernel_decode_attn(q.data_ptr(), pool_l.data_ptr(), pool_l.stride(0), block_table.data_ptr(),
                                          block_table.shape[1], plens, T, B, nq, nkv, dh, ps, pages, out.data_ptr(),
                                          scratch.data_ptr(), scratch.numel(), status.data_ptr(),
                                          torch.cuda.current_stream().cuda_stream))
    return out, status


def kernel_decode_attn_e4m3(q, codes_l, scales_l, block_table, kv_len, *, nq, nkv, ps, impl=0):
    """q bf16 [T, B, nq*128]; codes_l uint8 [T, pages, 2, nkv, ps, 128]; scales_l fp32 [T, pages, 2, nkv, ps];
    block_table int32 [B, maxp] (CUDA); kv_len: host ints [B]; impl 0 = tcgen05 kernel, 1 = mma.sync kernel.
    Returns (out bf16 [T, B, nq*128], status int32[16])."""
    import torch
    T, B, _ = q.shape
    pages = codes_l.shape[1]
    assert q.is_contiguous() and codes_l.is_contiguous() and scales_l.is_contiguous() and block_table.is_contiguous()
    assert q.dtype == torch.bfloat16 and codes_l.dtype == torch.uint8 and scales_l.dtype == torch.float32
    assert block_table.dtype == torch.int32 and tuple(scales_l.shape) == tuple(codes_l.shape[:-1])
    out = torch.empty_like(q)
    status = torch.zeros(16, dtype=torch.int32, device=q.device)
    n = _SZ()
    check(lib().pt_kernel_decode_attn_scratch_bytes(T, B, nq, 128, C.byref(n)))
    scratch = torch.empty(n.value, dtype=torch.uint8, device=q.device)
    lens, plens = _i32arr(kv_len)
    with torch.cuda.device(q.device):
        check(lib().pt_kernel_decode_attn_e4m3(q.data_ptr(), codes_l.data_ptr(), codes_l.stride(0), scales_l.data_ptr(),
                                               scales_l.stride(0), block_table.data_ptr(), block_table.shape[1], plens,
                                               T, B, nq, nkv, ps, pages, out.data_ptr(), impl, scratch.data_ptr(),
                                               scratch.numel(), status.data_ptr(), torch.cuda.current_stream().cuda_stream))
    return out, status


def kernel_prefill_attn(q, pool_l, block_table, kv_len, *, S, nq, nkv, dh, ps, impl=0):
    """q bf16 [T, B*S, nq*dh]; pool_l bf16 [T, pages, 2, nkv, ps, dh]; block_table int32 [B, maxp] and kv_len
    int32 [B] on the device (keys cached per sequence, the S new ones included).
    Returns (out bf16 [T, B*S, nq*dh], status int32[16])."""
    import torch
    T, M, _ = q.shape
    B = M // S
    assert q.is_contiguous() and pool_l.is_contiguous() and block_table.is_contiguous() and kv_len.is_cuda
    assert q.dtype == pool_l.dtype == torch.bfloat16 and block_table.dtype == kv_len.dtype == torch.int32
    out = torch.empty_like(q)
    status = torch.zeros(16, dtype=torch.int32, device=q.device)
    with torch.cuda.device(q.device):
        check(lib().pt_kernel_prefill_attn(q.data_ptr(), pool_l.data_ptr(), pool_l.stride(0), block_table.data_ptr(),
                                           block_table.shape[1], kv_len.data_ptr(), T, B, S, nq, nkv, dh, ps, pool_l.shape[1],
                                           out.data_ptr(), impl, status.data_ptr(), torch.cuda.current_stream().cuda_stream))
    return out, status


def kernel_decode_attn_static(q, pool_l, block_table, kv_len, *, nq, nkv, dh, ps, out=None, status=None):
    """pt_kernel_decode_attn for callers that may not allocate device memory: the scratch is an
    8 MiB array built into the library.  Pass preallocated ``out`` / ``status`` tensors to keep the
    call itself free of allocations; calls on one device must not overlap on the GPU."""
    import torch
    T, B, _ = q.shape
    if out is None:
        out = torch.empty_like(q)
    if status is None:
        status = torch.zeros(16, dtype=torch.int32, device=q.device)
    lens, plens = _i32arr(kv_len)
    with torch.cuda.device(q.device):
        check(lib().pt_kernel_decode_attn_static(q.data_ptr(), pool_l.data_ptr(), pool_l.stride(0), block_table.data_ptr(),
                                                 block_table.shape[1], plens, T, B, nq, nkv, dh, ps, pool_l.shape[1],
                                                 out.data_ptr(), status.data_ptr(), torch.cuda.current_stream().cuda_stream))
    return out, status
