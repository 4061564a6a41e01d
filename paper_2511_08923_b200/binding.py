"""ctypes binding of libtidar.so: argument marshalling only.

Every step of the decode path runs inside the library's CUDA kernels; this
module converts Python/torch objects into the plain pointers and sizes of the
C ABI declared in include/tidar.h, and keeps the borrowed device buffers alive.
PyTorch is used for device memory and the CUDA stream, nothing else.  If the
library cannot be loaded the import of :func:`load` fails loudly; there is no
CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np
import torch

from . import build as _build

TIDAR_OK = 0
ERR_NAMES = {-1: "TIDAR_EINVAL", -2: "TIDAR_ECAPACITY", -3: "TIDAR_ENOMEM", -4: "TIDAR_ECUDA", -5: "TIDAR_EDEVICE_TIMEOUT"}
TC_NAMES = ["embed", "norm", "gemm", "rope", "attn", "lmhead", "verify"]


class TidarError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"{ERR_NAMES.get(code, code)}: {msg}")
        self.code = code


class tidar_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab",
                                         "tie_lm_head")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)] + \
               [(n, C.c_int32) for n in ("mask_token_id", "k_max", "max_batch", "max_seq_len", "page_size")] + \
               [("beta", C.c_float), ("temperature", C.c_float), ("sample_seed", C.c_uint64),
                ("debug", C.c_int32), ("impl", C.c_int32), ("prefill_rows", C.c_int32)]


class tidar_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down",
                                                     "bqkv", "q_norm", "k_norm")]


_lib = None


def load(rebuild: bool = False) -> C.CDLL:
    """Build (if stale) and load libtidar.so; declare every prototype."""
    global _lib
    if _lib is not None and not rebuild:
        return _lib
    path = _build.build()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: the CUDA library must be built (there is no fallback)")
    lib = C.CDLL(path)
    P, I32, VP = C.POINTER, C.c_int32, C.c_void_p
    ctxp = VP
    sig = {
        "tidar_arena_bytes": (C.c_int, [P(tidar_config), P(C.c_size_t)]),
        "tidar_init": (C.c_int, [P(tidar_config), P(tidar_weights), VP, C.c_size_t, VP, P(ctxp)]),
        "tidar_prefill": (C.c_int, [ctxp, I32, P(I32), I32, I32, P(I32)]),
        "tidar_step": (C.c_int, [ctxp, P(I32), I32, P(I32), P(I32), P(I32)]),
        "tidar_step_async": (C.c_int, [ctxp, P(I32), I32, P(I32)]),
        "tidar_step_wait": (C.c_int, [ctxp, P(I32), P(I32)]),
        "tidar_step_k": (C.c_int, [ctxp, P(I32), I32, I32, P(I32), P(I32), P(I32)]),
        "tidar_step_ks": (C.c_int, [ctxp, P(I32), I32, P(I32), P(I32), P(I32), P(I32)]),
        "tidar_plan_ks": (C.c_int, [I32, I32, I32, P(I32), P(I32)]),
        "tidar_release": (C.c_int, [ctxp, I32]),
        "tidar_ar_step": (C.c_int, [ctxp, P(I32), I32, P(I32)]),
        "tidar_ridge_k": (C.c_int, [ctxp, I32, I32]),
        "tidar_score": (C.c_int, [ctxp, I32, P(I32), I32, P(C.c_float)]),
        "tidar_free": (C.c_int, [ctxp]),
        "tidar_last_error": (C.c_char_p, [ctxp]),
        "tidar_seq_len": (C.c_int, [ctxp, I32]),
        "tidar_launch_count": (C.c_int64, [ctxp]),
        "tidar_debug_set_block": (C.c_int, [ctxp, I32, P(I32)]),
        "tidar_debug_get_block": (C.c_int, [ctxp, I32, P(I32)]),
        "tidar_debug_last_rows": (C.c_int, [ctxp, P(I32), P(I32)]),
        "tidar_debug_get_logits": (C.c_int, [ctxp, I32, I32, P(C.c_float)]),
        "tidar_debug_get_hidden": (C.c_int, [ctxp, I32, I32, I32, P(C.c_float)]),
        "tidar_debug_get_argmax": (C.c_int, [ctxp, I32, I32, P(I32)]),
        "tidar_debug_get_kv": (C.c_int, [ctxp, I32, I32, I32, I32, P(C.c_uint16), P(C.c_uint16)]),
        "tidar_debug_set_timing": (C.c_int, [ctxp, I32]),
        "tidar_debug_get_timing": (C.c_int, [ctxp, P(C.c_float)]),
        "tidar_attention": (C.c_int, [ctxp, VP, VP, VP, I32, VP, I32, VP, VP, VP, VP, I32, I32]),
        "tidar_gemm": (C.c_int, [ctxp, VP, VP, I32, I32, I32, I32, VP]),
        "tidar_sync": (C.c_int, [ctxp]),
        "tidar_attention_static": (C.c_int, [VP, VP, VP, I32, VP, I32, VP, VP, VP, VP, I32, I32, I32, I32, I32, VP]),
        "tidar_debug_force_status": (C.c_int, [ctxp, I32]),
        "tidar_debug_wait_probe": (C.c_int, [ctxp, I32]),
        "tidar_debug_count_attention_tiles": (C.c_int, [ctxp, I32, P(C.c_uint64)]),
        "tidar_debug_set_timeline": (C.c_int, [ctxp, I32]),
        "tidar_debug_get_timeline": (C.c_int, [ctxp, P(C.c_float), P(C.c_float), P(C.c_float)]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _ip(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def pack_weights(w: dict, device) -> dict:
    """Arrange a generator-style weight dict in the layouts the C ABI asks for.

    Pure data movement: Q/K/V rows concatenated, gate/up rows interleaved
    (row 2f = gate f, row 2f+1 = up f), everything contiguous bf16 on ``device``.
    """
    def dev(x):
        return x.to(device=device, dtype=torch.bfloat16).contiguous()
    out = {"embed": dev(w["embed"]), "final_norm": dev(w["final_norm"])}
    out["lm_head"] = out["embed"] if w["lm_head"] is w["embed"] else dev(w["lm_head"])
    out["layers"] = []
    for L in w["layers"]:
        gu = torch.stack([L["w_gate"], L["w_up"]], dim=1).reshape(2 * L["w_gate"].shape[0], L["w_gate"].shape[1])
        lay = {
            "attn_norm": dev(L["attn_norm"]), "ffn_norm": dev(L["ffn_norm"]),
            "wqkv": dev(torch.cat([L["wq"], L["wk"], L["wv"]], dim=0)),
            "wo": dev(L["wo"]), "w_gate_up": dev(gu), "w_down": dev(L["w_down"]),
        }
        if "bq" in L:
            lay["bqkv"] = dev(torch.cat([L["bq"], L["bk"], L["bv"]], dim=0))
        if "q_norm" in L:
            lay["q_norm"], lay["k_norm"] = dev(L["q_norm"]), dev(L["k_norm"])
        out["layers"].append(lay)
    return out


class Tidar:
    """One library context: model weights + KV arena on one GPU."""

    def __init__(self, shape, packed: dict, k_max: int, max_batch: int = 1, max_seq_len: int = 4096,
                 debug: int = 0, impl: int = 0, device="cuda:0", stream: Optional[torch.cuda.Stream] = None,
                 guard_bytes: int = 0, beta: float = 1.0, prefill_rows: int = 0, temperature: float = 0.0, sample_seed: int = 0):
        self.lib = load()
        self.shape, self.k_max, self.max_batch = shape, k_max, max_batch
        self._async_n = []                   # listed sequences of the steps in flight, oldest first
        self.device = torch.device(device)
        cfg = tidar_config(
            n_layers=len(packed["layers"]), d_model=shape.d_model, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
            head_dim=shape.head_dim, d_ffn=shape.d_ffn, vocab=shape.vocab, tie_lm_head=int(shape.tie_lm_head),
            rms_eps=shape.rms_eps, rope_theta=shape.rope_theta, mask_token_id=shape.mask_token_id, k_max=k_max,
            max_batch=max_batch, max_seq_len=max_seq_len, page_size=64, beta=beta, temperature=temperature, sample_seed=sample_seed,
            debug=debug, impl=impl, prefill_rows=prefill_rows)
        self.cfg = cfg
        nbytes = C.c_size_t(0)
        rc = self.lib.tidar_arena_bytes(C.byref(cfg), C.byref(nbytes))
        if rc:
            raise TidarError(rc, (self.lib.tidar_last_error(None) or b"").decode())
        # guard_bytes > 0: a sentinel-filled tail right behind the arena (the library is told
        # nothing about it), so that a write past the arena can be detected: arena_guard_intact()
        self._guard_bytes = int(guard_bytes)
        with torch.cuda.device(self.device):
            self.arena = torch.empty(nbytes.value + 256 + self._guard_bytes, dtype=torch.uint8, device=self.device)
        base = (self.arena.data_ptr() + 255) // 256 * 256
        self._guard_off = base - self.arena.data_ptr() + nbytes.value
        if self._guard_bytes:
            self.arena[self._guard_off:].fill_(0xA5)
        self._packed = packed                     # keep the borrowed tensors alive
        nl = len(packed["layers"])
        arrs = {}
        for name in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down"):
            arrs[name] = (C.c_void_p * nl)(*[L[name].data_ptr() for L in packed["layers"]])
        for name in ("bqkv", "q_norm", "k_norm"):          # optional: present in every layer or in none
            if nl and name in packed["layers"][0]:
                arrs[name] = (C.c_void_p * nl)(*[L[name].data_ptr() for L in packed["layers"]])
        self._arrs = arrs
        wts = tidar_weights(embed=packed["embed"].data_ptr(), lm_head=packed["lm_head"].data_ptr(),
                            final_norm=packed["final_norm"].data_ptr(),
                            **{k: C.cast(v, C.POINTER(C.c_void_p)) for k, v in arrs.items()})
        self.stream = stream
        sh = C.c_void_p(stream.cuda_stream if stream is not None else 0)
        ctx = C.c_void_p()
        with torch.cuda.device(self.device):
            rc = self.lib.tidar_init(C.byref(cfg), C.byref(wts), C.c_void_p(base), C.c_size_t(nbytes.value), sh, C.byref(ctx))
        if rc:
            raise TidarError(rc, (self.lib.tidar_last_error(None) or b"").decode())
        self.ctx = ctx
        self.arena_bytes = nbytes.value

    # -- helpers -----------------------------------------------------------
    def _check(self, rc: int):
        if rc:
            raise TidarError(rc, (self.lib.tidar_last_error(self.ctx) or b"").decode())

    def arena_guard_intact(self) -> bool:
        """True if nothing wrote into the sentinel tail behind the arena (guard_bytes > 0)."""
        if not self._guard_bytes:
            return True
        torch.cuda.synchronize(self.device)
        return bool((self.arena[self._guard_off:] == 0xA5).all())

    def close(self):
        if getattr(self, "ctx", None):
            self.lib.tidar_free(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the path ------------------------------------------------------------
    def prefill(self, seq: int, prompt: Sequence[int], k: int) -> int:
        p = _i32(prompt)
        first = C.c_int32(0)
        self._check(self.lib.tidar_prefill(self.ctx, seq, _ip(p), len(p), k, C.byref(first)))
        return int(first.value)

    def step(self, seqs: Sequence[int], forced: Optional[Sequence[int]] = None):
        s = _i32(seqs)
        f = _i32(forced) if forced is not None else None
        toks = np.empty((len(s), self.k_max), dtype=np.int32)
        n = np.empty(len(s), dtype=np.int32)
        self._check(self.lib.tidar_step(self.ctx, _ip(s), len(s), _ip(f) if f is not None else None, _ip(toks), _ip(n)))
        return [toks[i, :n[i]].tolist() for i in range(len(s))], n.tolist()

    def step_k(self, seqs: Sequence[int], k: int, forced: Optional[Sequence[int]] = None):
        """A decode step with block length k chosen for this step (see tidar_step_k)."""
        s = _i32(seqs)
        f = _i32(forced) if forced is not None else None
        toks = np.empty((len(s), self.k_max), dtype=np.int32)
        n = np.empty(len(s), dtype=np.int32)
        self._check(self.lib.tidar_step_k(self.ctx, _ip(s), len(s), k, _ip(f) if f is not None else None, _ip(toks), _ip(n)))
        return [toks[i, :n[i]].tolist() for i in range(len(s))], n.tolist()

    def step_ks(self, seqs: Sequence[int], ks: Sequence[int], forced: Optional[Sequence[int]] = None):
        """A decode step in which each listed sequence uses its own block length (see tidar_step_ks)."""
        s = _i32(seqs)
        kk = _i32(ks)
        if len(kk) != len(s):
            raise ValueError("one block length per listed sequence")
        f = _i32(forced) if forced is not None else None
        toks = np.empty((len(s), self.k_max), dtype=np.int32)
        n = np.empty(len(s), dtype=np.int32)
        self._check(self.lib.tidar_step_ks(self.ctx, _ip(s), len(s), _ip(kk), _ip(f) if f is not None else None, _ip(toks), _ip(n)))
        return [toks[i, :n[i]].tolist() for i in range(len(s))], n.tolist()

    def release(self, seq: int):
        """Gives a sequence slot's KV pages back (see tidar_release)."""
        self._check(self.lib.tidar_release(self.ctx, seq))

    def ar_step(self, seqs: Sequence[int]) -> List[int]:
        """One plain autoregressive step: one new token per sequence (see tidar_ar_step)."""
        s = _i32(seqs)
        out = np.empty(len(s), dtype=np.int32)
        self._check(self.lib.tidar_ar_step(self.ctx, _ip(s), len(s), _ip(out)))
        return out.tolist()

    def ridge_k(self, n_seqs: int, row_budget: int = 0) -> int:
        return int(self.lib.tidar_ridge_k(self.ctx, n_seqs, row_budget))

    def score(self, seq: int, ids: Sequence[int]) -> np.ndarray:
        """log p(ids[i+1] | ids[..i]) for i in [0, n-1) from one causal pass (see tidar_score)."""
        a = _i32(ids)
        out = np.empty(len(a) - 1, dtype=np.float32)
        self._check(self.lib.tidar_score(self.ctx, seq, _ip(a), len(a), out.ctypes.data_as(C.POINTER(C.c_float))))
        return out

    def step_async(self, seqs: Sequence[int], forced: Sequence[int]):
        """Enqueues a step and returns; up to two may be in flight (see tidar_step_async)."""
        s, f = _i32(seqs), _i32(forced)
        self._check(self.lib.tidar_step_async(self.ctx, _ip(s), len(s), _ip(f)))
        self._async_n.append(len(s))

    def step_wait(self):
        """Results of the oldest step in flight (see tidar_step_wait)."""
        m = self._async_n[0] if self._async_n else self.max_batch
        toks = np.empty((m, self.k_max), dtype=np.int32)
        n = np.empty(m, dtype=np.int32)
        self._check(self.lib.tidar_step_wait(self.ctx, _ip(toks), _ip(n)))
        self._async_n.pop(0)
        return [toks[i, :n[i]].tolist() for i in range(m)], n.tolist()

    def seq_len(self, seq: int) -> int:
        rc = self.lib.tidar_seq_len(self.ctx, seq)
        if rc < 0:
            self._check(rc)
        return rc

    def launch_count(self) -> int:
        return int(self.lib.tidar_launch_count(self.ctx))

    # -- debug ---------------------------------------------------------------
    def set_block(self, seq: int, block: Sequence[int]):
        b = _i32(block)
        self._check(self.lib.tidar_debug_set_block(self.ctx, seq, _ip(b)))

    def get_block(self, seq: int, k: int) -> List[int]:
        b = np.empty(k, dtype=np.int32)
        self._check(self.lib.tidar_debug_get_block(self.ctx, seq, _ip(b)))
        return b.tolist()

    def last_rows(self):
        n, p = C.c_int32(0), C.c_int32(0)
        self._check(self.lib.tidar_debug_last_rows(self.ctx, C.byref(n), C.byref(p)))
        return int(n.value), int(p.value)

    def logits(self, row0: int, n_rows: int) -> np.ndarray:
        out = np.empty((n_rows, self.shape.vocab), dtype=np.float32)
        self._check(self.lib.tidar_debug_get_logits(self.ctx, row0, n_rows, out.ctypes.data_as(C.POINTER(C.c_float))))
        return out

    def hidden(self, layer: int, row0: int, n_rows: int) -> np.ndarray:
        out = np.empty((n_rows, self.shape.d_model), dtype=np.float32)
        self._check(self.lib.tidar_debug_get_hidden(self.ctx, layer, row0, n_rows, out.ctypes.data_as(C.POINTER(C.c_float))))
        return out

    def argmax(self, row0: int, n_rows: int) -> np.ndarray:
        out = np.empty(n_rows, dtype=np.int32)
        self._check(self.lib.tidar_debug_get_argmax(self.ctx, row0, n_rows, _ip(out)))
        return out

    def kv(self, seq: int, layer: int, pos0: int, npos: int):
        """(K, V) bf16 bit patterns as uint16 arrays [npos][n_kv_heads][head_dim]."""
        shp = (npos, self.shape.n_kv_heads, self.shape.head_dim)
        k, v = np.empty(shp, dtype=np.uint16), np.empty(shp, dtype=np.uint16)
        P16 = C.POINTER(C.c_uint16)
        self._check(self.lib.tidar_debug_get_kv(self.ctx, seq, layer, pos0, npos, k.ctypes.data_as(P16), v.ctypes.data_as(P16)))
        return k, v

    def wait_probe(self, limit_polls: int = 1 << 14):
        """Enqueue a kernel whose bounded wait runs out (see tidar_debug_wait_probe)."""
        self._check(self.lib.tidar_debug_wait_probe(self.ctx, int(limit_polls)))

    def force_status(self, value: int):
        """Test hook: pretend a kernel's bounded wait gave up (see tidar_debug_force_status)."""
        self._check(self.lib.tidar_debug_force_status(self.ctx, int(value)))

    def count_attention_tiles(self, on: bool) -> int:
        """Key tiles the attention kernel visited since the last call; sets the counter's switch."""
        v = C.c_uint64(0)
        self._check(self.lib.tidar_debug_count_attention_tiles(self.ctx, int(on), C.byref(v)))
        return int(v.value)

    def set_timeline(self, on: bool):
        self._check(self.lib.tidar_debug_set_timeline(self.ctx, int(on)))

    def timeline(self) -> dict:
        """Per-class kernel time (ms) of the last step from in-kernel stamps, plus 'busy' and 'span'."""
        ms = (C.c_float * len(TC_NAMES))()
        busy, span = C.c_float(0), C.c_float(0)
        self._check(self.lib.tidar_debug_get_timeline(self.ctx, ms, C.byref(busy), C.byref(span)))
        out = {n: float(ms[i]) for i, n in enumerate(TC_NAMES)}
        out["busy"], out["span"] = float(busy.value), float(span.value)
        return out

    def set_timing(self, on: bool):
        self._check(self.lib.tidar_debug_set_timing(self.ctx, int(on)))

    def timing(self) -> dict:
        ms = (C.c_float * len(TC_NAMES))()
        self._check(self.lib.tidar_debug_get_timing(self.ctx, ms))
        return {n: float(ms[i]) for i, n in enumerate(TC_NAMES)}

    def gemm(self, A, W, out, splits: int = 0):
        """out[R][N] (fp32) = A[R][K] @ W[N][K]^T on caller-owned device tensors (see tidar.h)."""
        R, K = A.shape
        N = W.shape[0]
        self._check(self.lib.tidar_gemm(self.ctx, A.data_ptr(), W.data_ptr(), R, N, K, splits, out.data_ptr()))

    def sync(self):
        self._check(self.lib.tidar_sync(self.ctx))

    def attention(self, q, k_pages, v_pages, page_table, seq_len, k_local, v_local, out, n_seqs: int, k: int):
        """Structured-mask attention alone, on caller-owned device tensors (see tidar.h)."""
        self._check(self.lib.tidar_attention(
            self.ctx, q.data_ptr(), k_pages.data_ptr(), v_pages.data_ptr(), k_pages.shape[0], page_table.data_ptr(), page_table.shape[1],
            seq_len.data_ptr(), k_local.data_ptr(), v_local.data_ptr(), out.data_ptr(), n_seqs, k))


def plan_ks(n_seqs: int, k_max: int, row_budget: int = 0, want: Optional[Sequence[int]] = None) -> List[int]:
    """Block lengths for one step of a batch under a budget of token slots (see tidar_plan_ks)."""
    lib = load()
    w = _i32(want) if want is not None else None
    if w is not None and len(w) != n_seqs:
        raise ValueError("one cap per sequence")
    out = np.empty(max(n_seqs, 1), dtype=np.int32)
    rc = lib.tidar_plan_ks(n_seqs, k_max, row_budget, _ip(w) if w is not None else None, _ip(out))
    if rc != 0:
        raise TidarError(rc, (lib.tidar_last_error(None) or b"").decode())
    return out[:n_seqs].tolist()


def attention_static(q, k_pages, v_pages, page_table, seq_len, k_local, v_local, out, n_seqs: int, k: int,
                     n_q_heads: int, n_kv_heads: int, head_dim: int, stream: Optional[torch.cuda.Stream] = None):
    """tidar_attention_static: the attention of a decode step for callers that cannot allocate.

    Needs no :class:`Tidar` context and no arena; all tensors are caller-owned device
    tensors in the layouts of :meth:`Tidar.attention`.  At most 4352 rows
    (``n_seqs * k * (k+1)``); calls that may overlap on the GPU must be serialised.
    """
    lib = load()
    rc = lib.tidar_attention_static(q.data_ptr(), k_pages.data_ptr(), v_pages.data_ptr(), k_pages.shape[0], page_table.data_ptr(),
                                    page_table.shape[1], seq_len.data_ptr(), k_local.data_ptr(), v_local.data_ptr(),
                                    out.data_ptr(), n_seqs, k, n_q_heads, n_kv_heads, head_dim,
                                    C.c_void_p(stream.cuda_stream if stream is not None else 0))
    if rc:
        raise TidarError(rc, (lib.tidar_last_error(None) or b"").decode())


def bf16_bits_to_f32(u16: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float32 values (exact)."""
    return (u16.astype(np.uint32) << 16).view(np.float32)
