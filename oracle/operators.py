"""TEST INFRASTRUCTURE ONLY -- the operators of a LLaMA block written as chains of scalar-keyed
join-aggs (paper Section 1: matmul, softmax, normalisation, elementwise maps and attention are
all a join followed by an aggregation).  fp64 inside; every store point rounds once, to the
nearest value of the stored relation's dtype (ties to even).

The paper does not print RMSNorm, SwiGLU or RoPE; the readings used here are listed in the
design notes (RMSNorm with eps inside the root, silu(t) = t / (1 + exp(-t)), RoPE on
interleaved pairs (2p, 2p+1) with positions counted from 0 in every sequence, softmax scale
1/sqrt(d_head)).  "parity unpinned" applies to two constants only: the value of eps and the
choice of the RoPE pairing; everything else is pinned by the CPU tests.
"""
from __future__ import annotations

import math

import numpy as np

from . import core


def rnd(a, dtype):
    return core.round_to(a, dtype) if dtype in ("f32", "bf16", "f16") else np.asarray(a, dtype=np.float64)


# ---- matmul -------------------------------------------------------------------------------------
def matmul(A, B, out_dtype="bf16"):
    """'ij,jk->ik', g = product, (+) = SUM (Example 3.4 / 3.8)."""
    return rnd(core.matmul(A, B), out_dtype)


# ---- SwiGLU MLP ---------------------------------------------------------------------------------
def silu_mul(a, b, out_dtype="bf16"):
    """'ij,ij->ij' key-aligned join, no aggregation: silu(a) * b."""
    return rnd(core.join_agg("ij,ij->ij", [a, b], fn="silu_mul", agg="none"), out_dtype)


def swiglu_mlp(x, W1, W3, W2, dtype="bf16"):
    a = matmul(x, W1, dtype)
    b = matmul(x, W3, dtype)
    h = silu_mul(a, b, dtype)
    y = matmul(h, W2, dtype)
    return {"a": a, "b": b, "h": h, "y": y}


# ---- RMSNorm ------------------------------------------------------------------------------------
def sumsq_rows(X):
    """'ij->i', g = square, (+) = SUM; statistics relation stored in fp32."""
    return rnd(core.join_agg("ij->i", [X], fn="square", agg="sum"), "f32")


def rms_scale(X, ss, gamma, eps, out_dtype="bf16"):
    """'ij,i,j->ij', g = x * (ss/n + eps)^(-1/2) * gamma, no aggregation."""
    n = np.shape(X)[1]
    return rnd(core.join_agg("ij,i,j->ij", [X, ss, gamma], fn="rms_scale", agg="none", params=(eps, float(n))),
               out_dtype)


def rmsnorm(X, gamma, eps=1e-5, out_dtype="bf16"):
    ss = sumsq_rows(X)
    return {"ss": ss, "y": rms_scale(X, ss, gamma, eps, out_dtype)}


# ---- row softmax --------------------------------------------------------------------------------
def softmax_rows(S, out_dtype="bf16"):
    """Over the last index of S[h,i,j]: MAX aggregation, then exp/SUM aggregation, then divide join."""
    m = rnd(core.join_agg("hij->hi", [S], fn="ident", agg="max"), "f32")
    l = rnd(core.join_agg("hij,hi->hi", [S, m], fn="exp_sub", agg="sum"), "f32")
    P = rnd(core.join_agg("hij,hi,hi->hij", [S, m, l], fn="exp_sub_div", agg="none"), out_dtype)
    return {"m": m, "l": l, "p": P}


# ---- attention ----------------------------------------------------------------------------------
def attention(Q, K, V, causal=True, out_dtype="bf16", scale=None, qpos=None):
    """[b,s,h,d] operands; plain definition, one rounding at the store of O."""
    scale = 1.0 / math.sqrt(np.shape(Q)[-1]) if scale is None else scale
    return rnd(core.attention(Q, K, V, scale, causal, qpos), out_dtype)


def attention_lse(Q, K, causal=True, scale=None, qpos=None):
    """Second output of the attention join-agg: lse[b,q,h] = log sum_k exp(scale * <Q[b,q,h,:], K[b,k,h,:]>) over the
    keys the query joins with (k <= q when causal).  With it two partial results over disjoint key ranges combine as
    O = w1 O1 + w2 O2, w_i = exp(lse_i - lse), lse = log(exp(lse_1) + exp(lse_2)) -- the online-softmax aggregation
    written for normalised partials.  Plain numpy route (independent of the C engine); statistics are stored in f32."""
    Q, K = np.asarray(Q, dtype=np.float64), np.asarray(K, dtype=np.float64)
    scale = 1.0 / math.sqrt(Q.shape[-1]) if scale is None else scale
    s = scale * np.einsum("bqhd,bkhd->bqhk", Q, K)
    if causal:
        pos = np.arange(Q.shape[1]) if qpos is None else np.asarray(qpos)
        s = np.where(np.arange(K.shape[1])[None, None, None, :] <= pos[None, :, None, None], s, -np.inf)
    m = s.max(axis=-1)
    some = np.isfinite(m)                         # a row that joins with no key: the sum is empty, its log is -inf
    ms = np.where(some, m, 0.0)
    with np.errstate(divide="ignore"):
        return rnd(np.where(some, ms + np.log(np.exp(s - ms[..., None]).sum(axis=-1)), -np.inf), "f32")


def attention_gqa_packed(Q, K, V, group=1, ends=None, causal=True, out_dtype="bf16", scale=None):
    """Grouped-query attention over packed sequences (Example 3.10). Q[b,s,hq,d], K,V[b,s,hkv,d] with hq = group*hkv:
    query heads [group*m, group*(m+1)) attend key/value head m; the sequence index holds independent sequences ending
    at `ends`, and attention never crosses a sequence boundary. Built from the plain definition above, one
    (sequence, query head) at a time."""
    Q, K, V = (np.asarray(t, dtype=np.float64) for t in (Q, K, V))
    B, S, Hq, D = Q.shape
    assert K.shape[2] * group == Hq
    ends = [S] if ends is None else list(ends)
    assert ends[-1] == S
    scale = 1.0 / math.sqrt(D) if scale is None else scale
    O = np.empty_like(Q)
    s0 = 0
    for s1 in ends:
        for h in range(Hq):
            g = h // group
            O[:, s0:s1, h:h + 1] = core.attention(Q[:, s0:s1, h:h + 1], K[:, s0:s1, g:g + 1], V[:, s0:s1, g:g + 1], scale, causal)
        s0 = s1
    return rnd(O, out_dtype)


def attention_as_join_aggs(Q, K, V, causal=True, scale=None):
    """The same operator as an explicit chain of scalar-keyed join-aggs (small shapes): scores =
    join on d + SUM; the causal band is a selection k <= q; MAX and exp/SUM aggregations over k;
    PV = join on k + SUM."""
    Q, K, V = (np.asarray(t, dtype=np.float64) for t in (Q, K, V))
    scale = 1.0 / math.sqrt(Q.shape[-1]) if scale is None else scale
    S = scale * core.join_agg("bqhd,bkhd->bhqk", [Q, K], fn="mul", agg="sum")
    pred = ("k", "q") if causal else None
    m = core.join_agg("bhqk->bhq", [S], fn="ident", agg="max", pred=pred)
    l = core.join_agg("bhqk,bhq->bhq", [S, m], fn="exp_sub", agg="sum", pred=pred)
    P = core.join_agg("bhqk,bhq,bhq->bhqk", [S, m, l], fn="exp_sub_div", agg="none")
    if causal:
        q_i, k_i = np.arange(S.shape[2])[:, None], np.arange(S.shape[3])[None, :]
        P = np.where(k_i <= q_i, P, 0.0)  # tuples removed by the selection contribute nothing to the SUM
    return core.join_agg("bhqk,bkhd->bqhd", [P, V], fn="mul", agg="sum")


def attention_combine(o_parts, lse_parts, out_dtype="bf16"):
    """The online-softmax aggregation of normalised partial attention results (O_c, lse_c) over disjoint key ranges:
    lse = log sum_c exp(lse_c), O = sum_c exp(lse_c - lse) O_c -- the (O~, m, l) combine of softmax_triple_combine with
    O_c = O~_c / l_c and lse_c = m_c + log l_c.  A partial with lse = -inf contributes nothing; a row without any key
    gets O = 0, lse = -inf.  Returns (O rounded once to out_dtype, lse rounded to f32), fp64 inside."""
    ls = np.stack([np.asarray(l, dtype=np.float64) for l in lse_parts])
    os_ = np.stack([np.asarray(o, dtype=np.float64) for o in o_parts])
    with np.errstate(divide="ignore", invalid="ignore"):
        mx = ls.max(axis=0)
        safe = np.where(np.isfinite(mx), mx, 0.0)
        tot = np.where(np.isfinite(mx), safe + np.log(np.exp(ls - safe).sum(axis=0)), -np.inf)
        w = np.where(np.isfinite(tot), np.exp(ls - np.where(np.isfinite(tot), tot, 0.0)), 0.0)
    O = np.where(w[..., None] > 0, w[..., None] * np.nan_to_num(os_), 0.0).sum(axis=0)   # an empty partial's O is never looked at
    return rnd(O, out_dtype), tot.astype(np.float32).astype(np.float64)


def softmax_triple_combine(a, b):
    """Online-softmax aggregation of two partial results (O~, m, l) of the same output key:
    m = max(m1, m2); O~ = O~1 e^(m1-m) + O~2 e^(m2-m); l = l1 e^(m1-m) + l2 e^(m2-m);
    identity (0, -inf, 0) with e^(-inf - -inf) := 0."""
    O1, m1, l1 = a
    O2, m2, l2 = b
    m = np.maximum(m1, m2)
    with np.errstate(invalid="ignore"):
        w1 = np.where(np.isneginf(m1), 0.0, np.exp(m1 - m))
        w2 = np.where(np.isneginf(m2), 0.0, np.exp(m2 - m))
    return O1 * w1[..., None] + O2 * w2[..., None], m, l1 * w1 + l2 * w2


def attention_blocked(Q, K, V, q_splits, k_splits, causal=True, scale=None):
    """Definition 3.7 for attention with the KV index split inside a sequence: one function
    specification per (b, h, q-block, k-block) that survives the band predicate; f returns the
    partial triple (O~, m, l) of its block pair; (+) is softmax_triple_combine; O = O~ / l."""
    Q, K, V = (np.asarray(t, dtype=np.float64) for t in (Q, K, V))
    B, S, H, D = Q.shape
    scale = 1.0 / math.sqrt(D) if scale is None else scale
    out = np.zeros_like(Q)
    for b in range(B):
        for h in range(H):
            for q0, q1 in zip(q_splits, q_splits[1:]):
                acc = (np.zeros((q1 - q0, D)), np.full(q1 - q0, -np.inf), np.zeros(q1 - q0))
                for k0, k1 in zip(k_splits, k_splits[1:]):
                    if causal and k0 > q1 - 1:
                        continue  # join predicate: no (q, k) pair of this block pair has k <= q
                    s = scale * core.join_agg("qd,kd->qk", [Q[b, q0:q1, h], K[b, k0:k1, h]])
                    if causal:
                        qi, ki = np.arange(q0, q1)[:, None], np.arange(k0, k1)[None, :]
                        s = np.where(ki <= qi, s, -np.inf)
                    m = s.max(axis=1)
                    with np.errstate(invalid="ignore"):
                        p = np.where(np.isneginf(s), 0.0, np.exp(s - np.where(np.isneginf(m), 0.0, m)[:, None]))
                    part = (core.join_agg("qk,kd->qd", [p, V[b, k0:k1, h]]), m, p.sum(axis=1))
                    acc = softmax_triple_combine(acc, part)
                out[b, q0:q1, h] = acc[0] / acc[2][:, None]
    return out


# ---- RoPE ---------------------------------------------------------------------------------------
def rope_rotation_relation(S, d, theta=1e4, pos=None):
    """R[s,p,c,e]: the 2x2 rotation by phi = t * theta^(-2p/d) for position t = pos[s] and pair p."""
    t = np.arange(S, dtype=np.float64) if pos is None else np.asarray(pos, dtype=np.float64)
    p = np.arange(d // 2, dtype=np.float64)
    phi = t[:, None] * theta ** (-2.0 * p / d)[None, :]
    R = np.empty((len(t), d // 2, 2, 2))
    R[..., 0, 0] = np.cos(phi); R[..., 0, 1] = -np.sin(phi)
    R[..., 1, 0] = np.sin(phi); R[..., 1, 1] = np.cos(phi)
    return R


def rope(x, theta=1e4, out_dtype="bf16", pos=None):
    """x[b,s,h,d] viewed as x[b,s,h,p,e] joined with R[s,p,c,e] on (s,p,e), SUM over e:
    (x[2p], x[2p+1]) <- (x[2p] cos - x[2p+1] sin, x[2p] sin + x[2p+1] cos)."""
    x = np.asarray(x, dtype=np.float64)
    B, S, H, D = x.shape
    R = rope_rotation_relation(S, D, theta, pos)
    y = core.join_agg("bshpe,spce->bshpc", [x.reshape(B, S, H, D // 2, 2), R], fn="mul", agg="sum")
    return rnd(y.reshape(B, S, H, D), out_dtype)


def add(x, y, out_dtype="bf16"):
    """'ij,ij->ij', g = sum, no aggregation (residual connection)."""
    return rnd(core.join_agg("ij,ij->ij", [x, y], fn="add", agg="none"), out_dtype)


# ---- LLaMA block --------------------------------------------------------------------------------
def llama_block(x, w, n_heads, theta=1e4, eps=1e-5, rows=None, dtype="bf16", n_kv_heads=None):
    """Pre-norm transformer block forward for ONE sequence x[S, hidden] (sequences of a batch are
    independent).  w: dict with wq, wo [hidden, hidden], wk, wv [hidden, n_kv_heads * d_head], w1, w3 [hidden, ffn],
    w2 [ffn, hidden], g1, g2 [hidden]; all weights are [in, out].  rows: optional subset of token positions for
    which the block output is wanted; K and V are always computed for the whole sequence.  With n_kv_heads <
    n_heads the attention is grouped-query (Example 3.10): query head h joins key/value head h // group."""
    x = np.asarray(x, dtype=np.float64)
    S, hidden = x.shape
    d = hidden // n_heads
    n_kv = n_heads if n_kv_heads is None else n_kv_heads
    group = n_heads // n_kv
    rows = np.arange(S) if rows is None else np.asarray(rows)
    n1 = rmsnorm(x, w["g1"], eps, dtype)["y"]
    k = matmul(n1, w["wk"], dtype)
    v = matmul(n1, w["wv"], dtype)
    q = matmul(n1[rows], w["wq"], dtype)
    k = rope(k.reshape(1, S, n_kv, d), theta, dtype)
    q = rope(q.reshape(1, len(rows), n_heads, d), theta, dtype, pos=rows)
    v4 = v.reshape(1, S, n_kv, d)
    att = np.empty((1, len(rows), n_heads, d))
    for hq in range(n_heads):     # plain definition, one query head at a time against its key/value head
        g = hq // group
        att[:, :, hq:hq + 1] = attention(q[:, :, hq:hq + 1], k[:, :, g:g + 1], v4[:, :, g:g + 1], causal=True, out_dtype=dtype, qpos=rows)
    att = att.reshape(len(rows), hidden)
    h = add(x[rows], matmul(att, w["wo"], dtype), dtype)
    n2 = rmsnorm(h, w["g2"], eps, dtype)["y"]
    y = swiglu_mlp(n2, w["w1"], w["w3"], w["w2"], dtype)["y"]
    out = add(h, y, dtype)
    return {"n1": n1, "q": q, "k": k, "v": v, "att": att, "h": h, "n2": n2, "mlp": y, "out": out}
