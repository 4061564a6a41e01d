"""CPU oracle for the TiDAR single-forward decode step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 NumPy statement of what the decode path computes,
written from the paper's description of the method.  Only the test suite, the
smoke check and the benchmark's CPU-baseline leg may use it; the CUDA library
shares no code with it and never calls it.

What the paper fixes and where (all citations are to the paper):

* Section 1 (what one generation step feeds the model): a step's forward
  carries the cached prefix, the tokens proposed by the previous step, and the
  mask-token slots that pre-draft the next step.
* Section 3.3 footnote: a step has ``q_len = k * (1 + k)`` token slots for a
  draft block of length ``k``: k causal slots followed by k blocks of k
  mask-token slots; the mask has shape ``(q_len, q_len + prefix)``.
* Figure "TiDAR Architecture" caption and Section 3.1: drafted tokens are
  encoded causally; mask tokens are bidirectional inside their block and see
  the prefix the block conditions on; KV of causally-forwarded tokens is stored
  and evicted for rejected tokens.
* Section 3.2: a draft survives iff it equals the autoregressive prediction
  computed in the current pass; pre-drafts exist for every acceptance outcome
  and the one matching the outcome is handed to the next step; generation
  starts with a causal prompt pass plus one bidirectional mask block
  (Appendix B, "Inference Prefill Mask").
* Section 4.4.3 (trusting AR vs diffusion): no label shift on mask slots, so the
  autoregressive output of causal slot b and the first slot of block b predict
  the same position; verification uses
  ``argmax(beta * logits_ar + (1 - beta) * logits_diff)``.

Readings taken where the paper is silent (listed again in the design notes):
mask slot (b, i) sits at position ``n + b + 1 + i``; block b sees causal slots
0..b; blocks do not see each other and causal slots see no mask slot; the first
causal slot is the token already settled by the previous pass, so acceptance
lengths run over 1..k; ties in argmax go to the lowest index.

Model family (the paper continues pre-training from Qwen2.5 and Qwen3 decoders,
Section 4.1): pre-norm decoder, RMSNorm, grouped-query attention with rotate-half
RoPE, SwiGLU FFN.  The two checkpoint families differ in two details, both optional
here and absent from the benchmark configurations: biases on the Q/K/V projections
(layer keys "bq", "bk", "bv") and an RMSNorm over each head's dimensions of Q and K
before RoPE (layer keys "q_norm", "k_norm").

parity pins: see tests/test_oracle_*.py.  Numeric values of hidden states and
logits have no printed example in the paper; they are pinned by a brute-force
per-row attention, by library routines (torch SDPA, a transformers Llama
decoder loaded with the same weights) and by the structural invariants.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------
# containers
# ----------------------------------------------------------------------------
@dataclass
class OracleConfig:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_theta: float
    rms_eps: float
    mask_token_id: int
    beta: float = 1.0
    # "f64": nothing is rounded (the definition).  "bf16": the activations a bf16 decoder keeps between
    # its operators (normed inputs of the projections, Q, K, V after RoPE, the attention output, the
    # SwiGLU output) are rounded to bfloat16 where they are stored; the paper trains and runs the
    # model in bfloat16 (Section 4.1).  All arithmetic stays float64 in both modes.
    act_dtype: str = "f64"
    # temperature 0: every prediction is the argmax (the hot path).  temperature > 0: every prediction is
    # a draw from softmax(logits / temperature), taken with noise that depends only on (sample_seed,
    # seq, predicted position, token id): see choose_tokens.
    temperature: float = 0.0
    sample_seed: int = 0
    seq: int = 0


@dataclass
class OracleState:
    """Sequence state between passes.

    ``n`` committed positions have K/V in ``k_cache[l]`` / ``v_cache[l]``
    (arrays ``[n, n_kv_heads, head_dim]``).  ``block`` is the next step's causal
    section: ``block[0]`` is the settled token at position n (already emitted),
    ``block[1:]`` are drafts for positions n+1 .. n+k-1.
    """
    n: int
    k_cache: List[np.ndarray]
    v_cache: List[np.ndarray]
    block: np.ndarray
    tokens: List[int] = field(default_factory=list)   # prompt + every emitted token


@dataclass
class ForwardOut:
    logits: np.ndarray              # [R, vocab]
    hidden: List[np.ndarray]        # input of each layer, then the final-norm input; [R, d]
    k_new: List[np.ndarray]         # per layer [R, n_kv_heads, head_dim] (after RoPE)
    v_new: List[np.ndarray]


def weights_to_f64(w: dict) -> dict:
    """Upcast a weight dict of array-likes (torch or numpy) to float64 NumPy."""
    def cv(x):
        if hasattr(x, "detach"):
            x = x.detach().to("cpu").float().numpy()
        return np.asarray(x, dtype=F64)
    out = {"embed": cv(w["embed"]), "final_norm": cv(w["final_norm"])}
    out["lm_head"] = out["embed"] if w["lm_head"] is w["embed"] else cv(w["lm_head"])
    out["layers"] = [{k: (v if k == "index" else cv(v)) for k, v in L.items()} for L in w["layers"]]
    return out


# ----------------------------------------------------------------------------
# masks  (Figure "TiDAR Attention Masks"; Section 3.3 footnote; Appendix B)
# ----------------------------------------------------------------------------
def n_slots(k: int) -> int:
    """Token slots in one decode step: k causal + k blocks of k mask slots."""
    return k * (1 + k)


def slot_layout(n: int, k: int):
    """Per-slot (kind, block, index-in-block, position) of a decode step.

    kind 0: causal slot j (position n + j).  kind 1: mask slot (b, i) at
    position n + b + 1 + i: with no label shift a mask slot predicts its own
    position, and block b starts right after causal slot b.
    """
    kind, blk, idx, pos = [], [], [], []
    for j in range(k):
        kind.append(0); blk.append(j); idx.append(0); pos.append(n + j)
    for b in range(k):
        for i in range(k):
            kind.append(1); blk.append(b); idx.append(i); pos.append(n + b + 1 + i)
    return (np.array(kind), np.array(blk), np.array(idx), np.array(pos, dtype=np.int64))


def build_decode_mask(n: int, k: int) -> np.ndarray:
    """Dense boolean mask [T, n + T] of a decode step, columns = [cache | step slots].

    Every row sees the whole committed prefix.  Causal slot j sees causal slots
    0..j and no mask slot.  Mask slot (b, i) sees causal slots 0..b (the prefix
    outcome block b conditions on) and the k slots of its own block.
    """
    T = n_slots(k)
    kind, blk, _, _ = slot_layout(n, k)
    m = np.zeros((T, n + T), dtype=bool)
    m[:, :n] = True
    for r in range(T):
        for c in range(T):
            if kind[r] == 0:
                ok = kind[c] == 0 and blk[c] <= blk[r]
            elif kind[c] == 0:
                ok = blk[c] <= blk[r]
            else:
                ok = blk[c] == blk[r]
            m[r, n + c] = ok
    return m


def build_prefill_mask(n: int, k: int) -> np.ndarray:
    """Dense boolean mask [(n + k), (n + k)] of the first pass.

    Prompt rows are causal; the k appended mask rows see the whole prompt and
    each other (one bidirectional block).
    """
    R = n + k
    m = np.zeros((R, R), dtype=bool)
    for r in range(R):
        for c in range(R):
            m[r, c] = (c <= r) if r < n else True
    m[:n, n:] = False
    return m


# ----------------------------------------------------------------------------
# layers
# ----------------------------------------------------------------------------
def round_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest bfloat16 (ties to even) of every element, returned as float64.

    bfloat16 is the upper half of an IEEE float32: the value is first taken to float32, then the low
    16 bits are rounded away (add 0x7FFF plus the lowest kept bit, clear the low half)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + (((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(F64)


def _stored(cfg: "OracleConfig", x: np.ndarray) -> np.ndarray:
    """An activation as the next operator reads it: unchanged, or rounded to bf16 (cfg.act_dtype)."""
    if cfg.act_dtype == "f64":
        return x
    assert cfg.act_dtype == "bf16", cfg.act_dtype
    return round_bf16(x)


def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotate-half RoPE.  x: [R, H, hd]; pair (i, i + hd/2) turns by pos * theta^(-2i/hd)."""
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = theta ** (-(np.arange(half, dtype=F64) * 2.0) / hd)
    ang = pos.astype(F64)[:, None] * inv_freq[None, :]          # [R, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def masked_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, mask: np.ndarray) -> np.ndarray:
    """softmax(q k^T / sqrt(hd) restricted to mask) v with grouped KV heads.

    q: [R, Hq, hd]; k, v: [C, Hkv, hd]; mask: [R, C] bool.  Query head h reads
    KV head h // (Hq / Hkv).  Returns [R, Hq, hd].
    """
    R, Hq, hd = q.shape
    Hkv = k.shape[1]
    g = Hq // Hkv
    out = np.empty_like(q)
    for h in range(Hq):
        s = (q[:, h, :] @ k[:, h // g, :].T) / np.sqrt(F64(hd))
        s = np.where(mask, s, -np.inf)
        s = s - s.max(axis=-1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=-1, keepdims=True)
        out[:, h, :] = p @ v[:, h // g, :]
    return out


def swiglu(gate: np.ndarray, up: np.ndarray) -> np.ndarray:
    return gate / (1.0 + np.exp(-gate)) * up


def forward(cfg: OracleConfig, w: dict, ids: np.ndarray, pos: np.ndarray, mask: np.ndarray,
            k_cache: Sequence[np.ndarray], v_cache: Sequence[np.ndarray],
            logit_rows: Optional[np.ndarray] = None) -> ForwardOut:
    """One transformer pass over R rows with an explicit dense mask.

    mask is [R, n_cache + R]: the first n_cache columns are the cached
    positions, the rest are this pass's own rows.  ``logit_rows`` restricts the
    LM head to some rows (others are returned as NaN) to bound oracle time.
    """
    R = len(ids)
    Hq, Hkv, hd = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    x = w["embed"][ids]                                          # [R, d]
    hidden, k_new, v_new = [], [], []
    for l, L in enumerate(w["layers"]):
        hidden.append(x.copy())
        a = _stored(cfg, rmsnorm(x, L["attn_norm"], cfg.rms_eps))
        q, kk, vv = a @ L["wq"].T, a @ L["wk"].T, a @ L["wv"].T
        if "bq" in L:                                   # projection biases (one checkpoint family)
            q, kk, vv = q + L["bq"], kk + L["bk"], vv + L["bv"]
        q, kk, vv = q.reshape(R, Hq, hd), kk.reshape(R, Hkv, hd), vv.reshape(R, Hkv, hd)
        if "q_norm" in L:                               # per-head RMSNorm of Q and K before RoPE (the other family)
            q, kk = rmsnorm(q, L["q_norm"], cfg.rms_eps), rmsnorm(kk, L["k_norm"], cfg.rms_eps)
        vv = _stored(cfg, vv)
        q = _stored(cfg, rope(q, pos, cfg.rope_theta))
        kk = _stored(cfg, rope(kk, pos, cfg.rope_theta))
        k_new.append(kk); v_new.append(vv)
        k_all = np.concatenate([k_cache[l], kk], axis=0) if len(k_cache[l]) else kk
        v_all = np.concatenate([v_cache[l], vv], axis=0) if len(v_cache[l]) else vv
        o = _stored(cfg, masked_attention(q, k_all, v_all, mask).reshape(R, Hq * hd))
        x = x + o @ L["wo"].T
        f = _stored(cfg, rmsnorm(x, L["ffn_norm"], cfg.rms_eps))
        x = x + _stored(cfg, swiglu(f @ L["w_gate"].T, f @ L["w_up"].T)) @ L["w_down"].T
    hidden.append(x.copy())
    y = _stored(cfg, rmsnorm(x, w["final_norm"], cfg.rms_eps))
    if logit_rows is None:
        logits = y @ w["lm_head"].T
    else:
        logits = np.full((R, cfg.vocab), np.nan, dtype=F64)
        logits[logit_rows] = y[logit_rows] @ w["lm_head"].T
    return ForwardOut(logits, hidden, k_new, v_new)


def argmax_lowest(x: np.ndarray) -> np.ndarray:
    """Row argmax; ties go to the lowest index (np.argmax does exactly that)."""
    return np.argmax(x, axis=-1)


# ----------------------------------------------------------------------------
# seeded sampling  (Section 3.2: drafts are sampled and then checked against the autoregressive
# prediction; read as token match, so "sampling" means: every prediction is a draw)
# ----------------------------------------------------------------------------
_M64 = (1 << 64) - 1


def mix64(z: int) -> int:
    """The output function of SplitMix64 (Steele, Lea, Flood 2014): a bijection of 64-bit words."""
    z &= _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def fmix32(h: np.ndarray) -> np.ndarray:
    """The 32-bit finaliser of MurmurHash3 (Appleby), element-wise on uint32."""
    h = h.astype(np.uint32)
    h ^= h >> np.uint32(16)
    h = (h * np.uint32(0x85EBCA6B)).astype(np.uint32)
    h ^= h >> np.uint32(13)
    h = (h * np.uint32(0xC2B2AE35)).astype(np.uint32)
    h ^= h >> np.uint32(16)
    return h


def position_key(seed: int, seq: int, pos: int) -> int:
    """32-bit key of one predicted position of one sequence: the top half of
    mix64(mix64(seed + golden ratio) ^ (seq << 32 | pos))."""
    return mix64(mix64(seed + 0x9E3779B97F4A7C15) ^ (((seq & 0xFFFFFFFF) << 32) | (pos & 0xFFFFFFFF))) >> 32


def gumbel_noise(seed: int, seq: int, pos: int, vocab: int) -> np.ndarray:
    """Standard Gumbel noise for every token id of one predicted position: u = (top 24 bits of
    fmix32(key + id * 0x9E3779B9) + 1/2) / 2^24 in (0, 1), noise = -log(-log(u))."""
    with np.errstate(over="ignore"):
        h = fmix32(np.uint32(position_key(seed, seq, pos)) + np.arange(vocab, dtype=np.uint32) * np.uint32(0x9E3779B9))
    u = ((h >> np.uint32(8)).astype(F64) + 0.5) * (1.0 / 16777216.0)
    return -np.log(-np.log(u))


def choose_tokens(cfg: OracleConfig, logits: np.ndarray, pred_pos: Sequence[int]) -> np.ndarray:
    """The model's prediction for each row: the argmax (temperature 0), or a draw from
    softmax(logits / temperature) by the Gumbel-max rule: argmax(logits / temperature + noise).

    The noise of a row depends on the POSITION the row predicts, not on the row: the autoregressive
    row of a position, the diffusion slots that pre-draft it and a plain one-token-per-pass decoder
    all draw with the same noise, so sampled TiDAR (beta = 1) emits exactly what sampled
    autoregressive decoding with this rule emits, and nothing depends on how positions are
    batched into passes."""
    logits = np.atleast_2d(logits)
    if cfg.temperature <= 0.0:
        return argmax_lowest(logits)
    out = np.empty(len(logits), dtype=np.int64)
    for r, p in enumerate(pred_pos):
        out[r] = int(np.argmax(logits[r] / cfg.temperature + gumbel_noise(cfg.sample_seed, cfg.seq, int(p), logits.shape[-1])))
    return out


# ----------------------------------------------------------------------------
# acceptance  (Section 3.2; Section 4.4.3)
# ----------------------------------------------------------------------------
def accept_length(block: Sequence[int], targets: Sequence[int], forced: int = 0) -> int:
    """Longest agreeing prefix.

    ``targets[j]`` is the verified prediction for position n + j + 1 made at
    causal slot j.  Draft ``block[i]`` (i >= 1) survives iff every earlier draft
    survived and ``block[i] == targets[i - 1]``.  The first slot is settled, so
    the result is in [1, k].  ``forced`` in [1, k] overrides the outcome (a
    benchmarking hook, not in the paper).
    """
    k = len(block)
    if forced:
        assert 1 <= forced <= k
        return int(forced)
    L = 1
    while L < k and int(block[L]) == int(targets[L - 1]):
        L += 1
    return L


def select_next(L: int, targets: Sequence[int], draft_ids: np.ndarray) -> np.ndarray:
    """Next causal section after accepting L slots.

    Its first token is the verified prediction at causal slot L-1 (the token for
    position n + L); the rest are the pre-drafts of block L-1, slots 1..k-1
    (positions n + L + 1 ...).  ``draft_ids`` is [k, k] = argmax of the mask
    slots' logits.
    """
    k = draft_ids.shape[0]
    nxt = np.empty(k, dtype=np.int64)
    nxt[0] = targets[L - 1]
    nxt[1:] = draft_ids[L - 1, 1:]
    return nxt


# ----------------------------------------------------------------------------
# passes
# ----------------------------------------------------------------------------
def _empty_cache(cfg: OracleConfig):
    z = np.zeros((0, cfg.n_kv_heads, cfg.head_dim), dtype=F64)
    return [z.copy() for _ in range(cfg.n_layers)], [z.copy() for _ in range(cfg.n_layers)]


def prefill(cfg: OracleConfig, w: dict, prompt: Sequence[int], k: int, return_forward: bool = False):
    """First pass: prompt rows causal plus one block of k mask rows (Appendix B).

    Row n-1 gives the autoregressive logits for position n; mask row i gives the
    diffusion logits for position n + i.  The settled first token mixes the two
    predictions of position n; the drafts are the argmax of mask rows 1..k-1.
    Only the prompt rows' K/V enter the cache.
    """
    n = len(prompt)
    ids = np.concatenate([np.asarray(prompt, dtype=np.int64), np.full(k, cfg.mask_token_id, dtype=np.int64)])
    pos = np.arange(n + k, dtype=np.int64)
    mask = build_prefill_mask(n, k)
    kc, vc = _empty_cache(cfg)
    rows = np.arange(n - 1, n + k)
    fo = forward(cfg, w, ids, pos, mask, kc, vc, logit_rows=None if return_forward else rows)
    a = fo.logits[n - 1]
    g = fo.logits[n:]
    c = int(choose_tokens(cfg, cfg.beta * a + (1.0 - cfg.beta) * g[0], [n])[0])      # row n-1 and mask row 0 predict position n
    block = np.empty(k, dtype=np.int64)
    block[0] = c
    block[1:] = choose_tokens(cfg, g[1:], n + np.arange(1, k))                        # mask row i predicts position n + i
    st = OracleState(n=n, k_cache=[x[:n].copy() for x in fo.k_new], v_cache=[x[:n].copy() for x in fo.v_new],
                     block=block, tokens=list(map(int, prompt)) + [c])
    return (st, c, fo) if return_forward else (st, c)


@dataclass
class StepOut:
    L: int
    emitted: List[int]
    targets: np.ndarray          # [k] verified predictions of the causal slots
    draft_ids: np.ndarray        # [k, k] argmax of every mask slot
    fwd: ForwardOut


def step(cfg: OracleConfig, w: dict, st: OracleState, forced: int = 0) -> StepOut:
    """One decode step: verify ``st.block`` and pre-draft every outcome in one pass."""
    k = len(st.block)
    n = st.n
    T = n_slots(k)
    _, _, _, pos = slot_layout(n, k)
    ids = np.concatenate([np.asarray(st.block, dtype=np.int64), np.full(k * k, cfg.mask_token_id, dtype=np.int64)])
    mask = build_decode_mask(n, k)
    fo = forward(cfg, w, ids, pos, mask, st.k_cache, st.v_cache)
    a = fo.logits[:k]                                  # causal slot j -> position n + j + 1
    g = fo.logits[k:].reshape(k, k, -1)                # mask (b, i) -> position n + b + 1 + i
    targets = choose_tokens(cfg, cfg.beta * a + (1.0 - cfg.beta) * g[:, 0, :], n + 1 + np.arange(k))
    draft_ids = choose_tokens(cfg, g.reshape(k * k, -1), [n + b + 1 + i for b in range(k) for i in range(k)]).reshape(k, k)
    L = accept_length(st.block, targets, forced)
    emitted = [int(t) for t in st.block[1:L]] + [int(targets[L - 1])]
    # commit K/V of the accepted causal slots only; the rest is evicted
    for l in range(cfg.n_layers):
        st.k_cache[l] = np.concatenate([st.k_cache[l], fo.k_new[l][:L]], axis=0)
        st.v_cache[l] = np.concatenate([st.v_cache[l], fo.v_new[l][:L]], axis=0)
    st.n = n + L
    st.block = select_next(L, targets, draft_ids)
    st.tokens.extend(emitted)
    return StepOut(L, emitted, targets, draft_ids, fo)


def generate(cfg: OracleConfig, w: dict, prompt: Sequence[int], k: int, max_new_tokens: int,
             draft_hook=None, forced: Optional[Sequence[int]] = None):
    """TiDAR generation: prefill, then steps until ``max_new_tokens`` are out.

    ``draft_hook(state)`` may overwrite ``state.block[1:]`` before each step (to
    test that the output does not depend on draft quality when beta = 1).
    Returns (new tokens, list of acceptance lengths, final state).
    """
    st, c = prefill(cfg, w, prompt, k)
    out = [c]
    Ls = []
    s = 0
    while len(out) < max_new_tokens:
        if draft_hook is not None:
            draft_hook(st)
        so = step(cfg, w, st, forced=int(forced[s]) if forced is not None else 0)
        out.extend(so.emitted)
        Ls.append(so.L)
        s += 1
    return out[:max_new_tokens], Ls, st


def causal_forward(cfg: OracleConfig, w: dict, ids: Sequence[int]) -> ForwardOut:
    """Plain causal pass over a whole sequence (the autoregressive definition)."""
    ids = np.asarray(ids, dtype=np.int64)
    R = len(ids)
    mask = np.tril(np.ones((R, R), dtype=bool))
    kc, vc = _empty_cache(cfg)
    return forward(cfg, w, ids, np.arange(R, dtype=np.int64), mask, kc, vc)


def ar_generate(cfg: OracleConfig, w: dict, prompt: Sequence[int], max_new_tokens: int) -> List[int]:
    """Greedy autoregressive decoding, one token per causal pass with a KV cache."""
    ids = np.asarray(prompt, dtype=np.int64)
    n = len(ids)
    kc, vc = _empty_cache(cfg)
    fo = forward(cfg, w, ids, np.arange(n, dtype=np.int64), np.tril(np.ones((n, n), dtype=bool)), kc, vc,
                 logit_rows=np.array([n - 1]))
    kc, vc = [x.copy() for x in fo.k_new], [x.copy() for x in fo.v_new]
    out = [int(choose_tokens(cfg, fo.logits[n - 1], [n])[0])]
    while len(out) < max_new_tokens:
        m = np.ones((1, n + 1), dtype=bool)
        fo = forward(cfg, w, np.array([out[-1]]), np.array([n], dtype=np.int64), m, kc, vc)
        for l in range(cfg.n_layers):
            kc[l] = np.concatenate([kc[l], fo.k_new[l]], axis=0)
            vc[l] = np.concatenate([vc[l], fo.v_new[l]], axis=0)
        n += 1
        out.append(int(choose_tokens(cfg, fo.logits[0], [n])[0]))
    return out
