"""CPU oracle for the shared-base + low-rank (LR) KV-cache path.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain definition that the CUDA kernels are checked
against.  It is imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg, never by the product path, and it shares no code with the
CUDA sources.  Everything is numpy float64; matrix products use ``@`` as a
library step and nothing is blocked, fused or reordered beyond what each
docstring states.

What it computes (paper notation, Section 2.1):

* Eq. 1: for agent i,  Y_i = X (W0 + A_i B_i) = X W0 + (X A_i) B_i.  The left
  form (merged weight) is the *definition* used for every expected value.  The
  right form (base cache X W0 plus LR cache X A_i, Section 2.2) exists here only
  so that the tests can check the two against each other.
* The benchmark's working form carries the usual LoRA scale s = alpha / r:
  W_eff = W0 + s A_i B_i.  s = 1 is Eq. 1 literally.
* Attention of the current agent over the shared context (Section 3.1): plain
  softmax attention with the agent's own adapted K and V, scale sigma = 1/sqrt(hd),
  grouped-query mapping q-head h -> kv-head h // (n_q / n_kv).  The main path is
  position-free.  The rotary variant (Appendix D.2: a rotated key needs the rank-r
  term expanded to full width before the rotation) is ``rope_rotate`` /
  ``lr_decode_reference_rope``: K_a[t] = RoPE_t(H_t (W_k + s A B)), rotate-half
  pairing (c, c + hd/2), angle t * theta^(-2c/hd); values are never rotated.
* Decode attends over exactly ``ctx_len`` cached tokens (the caller has already
  appended the current token).  New-turn prefill of S tokens that sit at
  positions T .. T+S-1: query i sees positions 0 .. T+i (context fully visible,
  causal among the new tokens).

Pins (tests/test_oracle_pins.py): r = 0 / B = 0 / s = 0 reduce to base-only
attention; merged == decomposed; softmax rows sum to one and outputs are convex
combinations of V rows; ctx_len = 1, q = 0 and identical-rows closed forms;
permutation invariance; prefill row i == decode at ctx T+i+1; agent isolation;
pure-Python float brute force on tiny shapes; the LR/base byte ratio against the
paper's memory table; for the rotary functions: norm preservation, identity at
position 0, dependence on relative position only, an explicit 2x2 rotation, the
linearity that makes expand-then-rotate equal the merged weight, and brute force.
No function here is unpinned.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def as_f64(x) -> np.ndarray:
    """Exact widening of an array-like (bf16 values held in fp32 are exact in fp64)."""
    return np.asarray(x, dtype=F64)


# --------------------------------------------------------------------------- Eq. 1

def merged_weight(W0, A, B, s: float) -> np.ndarray:
    """W_eff = W0 + s * A B  (Eq. 1, left form, with the LoRA scale s)."""
    W0, A, B = as_f64(W0), as_f64(A), as_f64(B)
    if A.shape[-1] == 0:
        return W0.copy()
    return W0 + s * (A @ B)


def adapted_projection(X, W0, A, B, s: float) -> np.ndarray:
    """Y = X (W0 + s A B)  (Eq. 1, left form): the agent's full-width K or V rows."""
    return as_f64(X) @ merged_weight(W0, A, B, s)


def base_cache(X, W0) -> np.ndarray:
    """Base contribution X W0 (Eq. 1; the shared base cache of Section 2.2)."""
    return as_f64(X) @ as_f64(W0)


def lr_cache(X, A) -> np.ndarray:
    """LR cache X A, width r (Section 2.2; built for every agent in Section 3.1)."""
    return as_f64(X) @ as_f64(A)


def decomposed_projection(X, W0, A, B, s: float) -> np.ndarray:
    """X W0 + s (X A) B  (Eq. 1, right form)."""
    return reconstruct(base_cache(X, W0), lr_cache(X, A), B, s)


def reconstruct(base, L, B, s: float) -> np.ndarray:
    """base + s L B : the adapted rows rebuilt from a base cache and an LR cache."""
    base, L, B = as_f64(base), as_f64(L), as_f64(B)
    if L.shape[-1] == 0:
        return base.copy()
    return base + s * (L @ B)


# ----------------------------------------------------------------------- attention

def softmax_weights(z: np.ndarray) -> np.ndarray:
    """Two-pass softmax of one row of logits."""
    z = as_f64(z)
    e = np.exp(z - np.max(z))
    return e / np.sum(e)


def attend_rows(q_h, K_g, V_g, sigma: float) -> np.ndarray:
    """softmax(sigma * K_g q_h) V_g for one query head over the given rows.

    q_h [hd], K_g [t, hd], V_g [t, hd] -> [hd].
    """
    p = softmax_weights(sigma * (as_f64(K_g) @ as_f64(q_h)))
    return p @ as_f64(V_g)


def _sigma(hd: int, sigma) -> float:
    return 1.0 / np.sqrt(hd) if sigma is None or sigma <= 0 else float(sigma)


def attend_decode_one(q, K, V, ctx_len: int, n_kv: int, sigma=None) -> np.ndarray:
    """Decode attention of one request.

    q [n_q, hd]; K, V [>=ctx_len, n_kv*hd] (that request's agent's adapted rows);
    attends over rows 0..ctx_len-1; q-head h uses kv-head h // (n_q/n_kv).
    Returns [n_q, hd].
    """
    q, K, V = as_f64(q), as_f64(K), as_f64(V)
    n_q, hd = q.shape
    G = n_q // n_kv
    sg = _sigma(hd, sigma)
    out = np.empty((n_q, hd), dtype=F64)
    for h in range(n_q):
        g = h // G
        out[h] = attend_rows(q[h], K[:ctx_len, g * hd:(g + 1) * hd], V[:ctx_len, g * hd:(g + 1) * hd], sg)
    return out


def attend_prefill(q, K, V, T: int, n_kv: int, sigma=None, rows=None) -> np.ndarray:
    """New-turn prefill attention.

    q [S, n_q, hd]; K, V [>=T+S, n_kv*hd]; query i attends rows 0..T+i.
    ``rows`` optionally restricts the computed query indices (others are NaN).
    Returns [S, n_q, hd].
    """
    q = as_f64(q)
    S = q.shape[0]
    out = np.full(q.shape, np.nan, dtype=F64)
    for i in (range(S) if rows is None else rows):
        out[i] = attend_decode_one(q[i], K, V, T + i + 1, n_kv, sigma)
    return out


# ------------------------------------------------------------ whole-path references

def lr_decode_reference(q, agent_id, ctx_len, H, W_k, W_v, A_k, B_k, A_v, B_v,
                        s_k: float, s_v: float, n_kv: int, sigma=None, heads=None) -> np.ndarray:
    """Decode over a shared context from first principles (merged weights).

    q [B, n_q, hd]; agent_id [B]; ctx_len [B]; H [T, d] shared by all requests;
    A_* [N, d, r], B_* [N, r, n_kv*hd].  For request b with agent a:
    K_a = H (W_k + s_k A_a^K B_a^K), V_a likewise, then ``attend_decode_one``.
    ``heads`` optionally restricts the kv-heads evaluated (others NaN) so that
    large cases can be sampled: only the sampled head's columns are projected.
    """
    q = as_f64(q)
    Bn, n_q, hd = q.shape
    G = n_q // n_kv
    out = np.full(q.shape, np.nan, dtype=F64)
    kv_heads = range(n_kv) if heads is None else heads
    H = as_f64(H)
    for b in range(Bn):
        a = int(agent_id[b])
        t = int(ctx_len[b])
        for g in kv_heads:
            cols = slice(g * hd, (g + 1) * hd)
            K = H[:t] @ merged_weight(as_f64(W_k)[:, cols], A_k[a], as_f64(B_k[a])[:, cols], s_k)
            V = H[:t] @ merged_weight(as_f64(W_v)[:, cols], A_v[a], as_f64(B_v[a])[:, cols], s_v)
            sg = _sigma(hd, sigma)
            for h in range(g * G, (g + 1) * G):
                out[b, h] = attend_rows(q[b, h], K, V, sg)
    return out


def lr_prefill_reference(q, agent: int, T: int, H, W_k, W_v, A_k, B_k, A_v, B_v,
                         s_k: float, s_v: float, n_kv: int, sigma=None, heads=None, rows=None) -> np.ndarray:
    """New-turn prefill from first principles; H [T+S, d] covers context + new tokens."""
    q = as_f64(q)
    S, n_q, hd = q.shape
    G = n_q // n_kv
    out = np.full(q.shape, np.nan, dtype=F64)
    H = as_f64(H)
    sg = _sigma(hd, sigma)
    for g in (range(n_kv) if heads is None else heads):
        cols = slice(g * hd, (g + 1) * hd)
        K = H[:T + S] @ merged_weight(as_f64(W_k)[:, cols], A_k[agent], as_f64(B_k[agent])[:, cols], s_k)
        V = H[:T + S] @ merged_weight(as_f64(W_v)[:, cols], A_v[agent], as_f64(B_v[agent])[:, cols], s_v)
        for i in (range(S) if rows is None else rows):
            for h in range(g * G, (g + 1) * G):
                out[i, h] = attend_rows(q[i, h], K[:T + i + 1], V[:T + i + 1], sg)
    return out


def attend_from_caches(q_b, k_base, v_base, L_k, L_v, B_k_a, B_v_a, s_k: float, s_v: float,
                       n_kv: int, sigma=None, heads=None) -> np.ndarray:
    """Attention of one request given cache *contents* (token-major rows).

    k_base, v_base [t, n_kv*hd]; L_k [t, r_k]; L_v [t, r_v]; B_*_a [r, n_kv*hd]
    of the request's agent.  K_a = k_base + s_k L_k B_k (Eq. 1, right form), V_a
    likewise; then plain attention over all t rows.  Used where a workload fills
    the caches directly instead of deriving them from hidden states.
    """
    q_b = as_f64(q_b)
    n_q, hd = q_b.shape
    G = n_q // n_kv
    out = np.full(q_b.shape, np.nan, dtype=F64)
    sg = _sigma(hd, sigma)
    for g in (range(n_kv) if heads is None else heads):
        cols = slice(g * hd, (g + 1) * hd)
        K = reconstruct(as_f64(k_base)[:, cols], L_k, as_f64(B_k_a)[:, cols], s_k)
        V = reconstruct(as_f64(v_base)[:, cols], L_v, as_f64(B_v_a)[:, cols], s_v)
        for h in range(g * G, (g + 1) * G):
            out[h] = attend_rows(q_b[h], K, V, sg)
    return out


# ------------------------------------------------------------ rotary keys (Appendix D.2)

def rope_tables(max_pos: int, hd: int, theta: float = 10000.0):
    """cos/sin tables [max_pos, hd/2] of the rotate-half rotary embedding: angle(t, c) = t * theta^(-2c/hd)."""
    inv = theta ** (-np.arange(hd // 2, dtype=F64) * 2.0 / hd)
    ang = np.arange(max_pos, dtype=F64)[:, None] * inv[None, :]
    return np.cos(ang), np.sin(ang)


def rope_rotate(x, pos, n_heads: int, cos, sin) -> np.ndarray:
    """Rotate rows x [t, n_heads*hd] head by head: coordinates (c, c + hd/2) of a head turn by the angle
    of the row's position (rotate-half convention: x' = x cos + rotate_half(x) sin)."""
    x = as_f64(x)
    t, w = x.shape
    hd = w // n_heads
    xs = x.reshape(t, n_heads, 2, hd // 2)
    c = as_f64(cos)[np.asarray(pos)][:, None, :]
    s_ = as_f64(sin)[np.asarray(pos)][:, None, :]
    lo, hi = xs[:, :, 0], xs[:, :, 1]
    out = np.stack([lo * c - hi * s_, hi * c + lo * s_], axis=2)
    return out.reshape(t, w)


def lr_decode_reference_rope(q, agent_id, ctx_len, H, W_k, W_v, A_k, B_k, A_v, B_v, s_k: float, s_v: float,
                             n_kv: int, cos, sin, sigma=None) -> np.ndarray:
    """Decode with rotary keys from first principles: the agent's key row of token t is
    RoPE_t(H_t (W_k + s_k A B)), i.e. the rank-r contribution is expanded to full width BEFORE the
    rotation (Appendix D.2); values are not rotated; q arrives already rotated.  Token t sits at position t."""
    q = as_f64(q)
    Bn, n_q, hd = q.shape
    out = np.empty(q.shape, dtype=F64)
    H = as_f64(H)
    for b in range(Bn):
        a, t = int(agent_id[b]), int(ctx_len[b])
        K = rope_rotate(H[:t] @ merged_weight(W_k, A_k[a], B_k[a], s_k), np.arange(t), n_kv, cos, sin)
        V = H[:t] @ merged_weight(W_v, A_v[a], B_v[a], s_v)
        out[b] = attend_decode_one(q[b], K, V, t, n_kv, sigma)
    return out


def lr_prefill_reference_rope(q, agent: int, T: int, H, W_k, W_v, A_k, B_k, A_v, B_v, s_k: float, s_v: float,
                              n_kv: int, cos, sin, sigma=None, rows=None) -> np.ndarray:
    """New-turn prefill with rotary keys from first principles: the agent's keys of all T + S tokens are
    RoPE_t(H_t (W_k + s_k A B)) (token t at position t), values un-rotated, then ``attend_prefill``."""
    q = as_f64(q)
    S = q.shape[0]
    H = as_f64(H)[:T + S]
    K = rope_rotate(H @ merged_weight(W_k, A_k[agent], B_k[agent], s_k), np.arange(T + S), n_kv, cos, sin)
    V = H @ merged_weight(W_v, A_v[agent], B_v[agent], s_v)
    return attend_prefill(q, K, V, T, n_kv, sigma, rows)


# ------------------------------------------------------------------ cache accounting

def cache_bytes_per_token(n_kv: int, hd: int, n_agents: int, rank_k: int, rank_v: int,
                          bytes_per_elem: int = 2):
    """(base bytes, LR bytes) one layer stores per context token.

    One shared base K and V row of width n_kv*hd, plus for every agent one LR row
    of width r per adapted projection (Sections 2.2 and 4.3, memory usage).
    """
    base = 2 * n_kv * hd * bytes_per_elem
    lr = n_agents * (rank_k + rank_v) * bytes_per_elem
    return base, lr
