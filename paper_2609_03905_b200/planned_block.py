"""A LLaMA-shaped transformer block executed under a plan of the logical optimizer (Section 4): one join-agg spec per
abstract operator, as `ja_plan_optimize_graph` returns it, and a `ja_repartition` exactly where a producer's output
tiling differs from the tiling the consumer's spec needs (sub-cost 1 of Section 4.3). Nothing here computes: the class
turns interval counts into split lists, relations and specs, and `forward()` is an ordered list of library calls.

The block is written on tensors `x[b, s, e]` (batch, sequence, hidden) and `q[b, s, h, d]` (heads, head dimension; `d` is
not shardable), as the graph of eleven abstract operators of `block_graph()`; the norm output, the post-attention residual
and the second norm output are consumed more than once (Section 4.5).

How a spec on `[b, s, ...]` tensors reaches kernels written for `[rows, columns]` relations: a relation `[b, s, e]` with
blocks `[bb, sb, eb]` stores every block as a dense `(bb * sb) x eb` matrix, blocks in key order -- byte for byte the
payload of a relation `[rows, e]` whose row blocks are the `(b-interval, s-interval)` pairs in key order. A contraction
over `e`, a row-wise norm or a key-aligned join does not care in which order the token rows are stored as long as every
operand uses the same order, so those operators run on such two-index views (second handles over the same payloads, no
copy). Relayouts, RoPE and attention run on the tensors' own indices.
"""
from __future__ import annotations

import math

import torch

from . import binding as B
from .relations import Relation, Spec, equal_splits as ES, from_dense, repartition


def block_graph(batch: int, seq: int, hidden: int, n_heads: int, ffn: int):
    """The block as the optimizer sees it: eleven abstract operators in topological order (RoPE is part of the q / k
    projections). `inputs`: producer index per operand, None for inputs of the computation (x, weights, gains)."""
    D = hidden // n_heads
    E = lambda **k: k
    return [
        {"einsum": "bse,e->bse", "extents": E(b=batch, s=seq, e=hidden), "inputs": [None, None]},                                   # 0 n1
        {"einsum": "bse,ehd->bshd", "extents": E(b=batch, s=seq, e=hidden, h=n_heads, d=D), "inputs": [0, None], "fixed": {"d"}},   # 1 q
        {"einsum": "bse,ehd->bshd", "extents": E(b=batch, s=seq, e=hidden, h=n_heads, d=D), "inputs": [0, None], "fixed": {"d"}},   # 2 k
        {"einsum": "bse,ehd->bshd", "extents": E(b=batch, s=seq, e=hidden, h=n_heads, d=D), "inputs": [0, None], "fixed": {"d"}},   # 3 v
        {"einsum": "bqhd,bkhd,bkhd->bqhd", "extents": E(b=batch, q=seq, h=n_heads, d=D, k=seq), "inputs": [1, 2, 3], "fixed": {"d"}},  # 4 att
        {"einsum": "bshd,hde,bse->bse", "extents": E(b=batch, s=seq, h=n_heads, d=D, e=hidden), "inputs": [4, None, None], "fixed": {"d"}},  # 5 h
        {"einsum": "bse,e->bse", "extents": E(b=batch, s=seq, e=hidden), "inputs": [5, None]},                                      # 6 n2
        {"einsum": "bse,ef->bsf", "extents": E(b=batch, s=seq, e=hidden, f=ffn), "inputs": [6, None]},                              # 7 a
        {"einsum": "bse,ef->bsf", "extents": E(b=batch, s=seq, e=hidden, f=ffn), "inputs": [6, None]},                              # 8 b
        {"einsum": "bsf,bsf->bsf", "extents": E(b=batch, s=seq, f=ffn), "inputs": [7, 8]},                                          # 9 silu(a) b
        {"einsum": "bsf,fe,bse->bse", "extents": E(b=batch, s=seq, f=ffn, e=hidden), "inputs": [9, None, 5]},                       # 10 out
    ]


def _terms(einsum: str):
    lhs, out = einsum.replace(" ", "").split("->")
    return lhs.split(","), out


class _Tensor:
    """One tensor of the block in one tiling: its relation over its own indices."""

    def __init__(self, letters: str, extents: dict, counts: dict, dtype=torch.bfloat16, dense: torch.Tensor | None = None):
        self.letters = letters
        self.ext = [extents[c] for c in letters]
        self.counts = tuple(counts[c] for c in letters)
        self.splits = [ES(e, n) for e, n in zip(self.ext, self.counts)]
        self.rel = from_dense(dense.reshape(self.ext), self.splits) if dense is not None else Relation(self.ext, self.splits, dtype)

    def rows_view(self, n_row_letters: int) -> Relation:
        """Two-index view: the first n_row_letters indices flattened into rows (blocks in key order), the rest into columns."""
        def flat(exts, splits):
            """Several indices as one: a block of the flattened index is one block per index, its size the product of their
            sizes, and blocks follow key order (first index slowest)."""
            sizes = [[]]
            for sp in splits:
                sizes = [a + [sp[i + 1] - sp[i]] for a in sizes for i in range(len(sp) - 1)]
            out = [0]
            for a in sizes:
                out.append(out[-1] + math.prod(a))
            return math.prod(exts), out
        r_ext, r_sp = flat(self.ext[:n_row_letters], self.splits[:n_row_letters])
        c_ext, c_sp = flat(self.ext[n_row_letters:], self.splits[n_row_letters:])
        # columns may only be flattened when all but the first column index are unsplit (else a block is not a dense matrix)
        assert all(n == 1 for n in self.counts[n_row_letters + 1:]), "only the first column index of a view may be split"
        return self.rel.view_as([r_ext, c_ext], [r_sp, c_sp])


class PlannedBlock:
    """counts: one {letter: intervals} dict per operator of block_graph(), e.g. the plan of ja_plan_optimize_graph."""

    def __init__(self, batch: int, seq: int, hidden: int, n_heads: int, ffn: int, weights: dict, counts, theta: float = 1e4,
                 eps: float = 1e-5, fused: bool = True, share_relayouts: bool = False, dtype: torch.dtype = torch.bfloat16):
        assert hidden // n_heads == 128, "the attention kernels need head dimension 128"
        self.B, self.S, self.hidden, self.H, self.ffn = batch, seq, hidden, n_heads, ffn
        self.T = batch * seq
        D = hidden // n_heads
        self.ops = block_graph(batch, seq, hidden, n_heads, ffn)
        self.counts = [dict(c) for c in counts]
        assert len(self.counts) == len(self.ops)
        for op, c in zip(self.ops, self.counts):
            assert c.get("d", 1) == 1, "the head dimension is not shardable"
        assert dtype in (torch.bfloat16, torch.float16)
        bf = self.dtype = dtype    # cell type of every relation of the block
        w = {n: weights[n].to("cuda", bf) for n in weights}
        ops, cn = self.ops, self.counts
        self.steps = []            # (name, callable) in execution order
        self.n_relayouts = 0       # relayouts of tensors produced inside the block = repartition charges of the plan
        self.n_input_relayouts = 0 # relayouts of the block input x (inputs of the computation are free in the cost model)

        def out_tensor(i):
            _, out = _terms(ops[i]["einsum"])
            return self._tensor(out, ops[i]["extents"], cn[i])
        self.out_t = [out_tensor(i) for i in range(len(ops))]

        def operand(i, k, dense=None, name=""):
            """Relation of operand k of operator i in the tiling in_k(J_i): the producer's output itself when the tilings
            agree, else a second relation filled by a relayout step scheduled right before the operator."""
            ins, _ = _terms(ops[i]["einsum"])
            term = ins[k]
            prod = ops[i]["inputs"][k]
            if prod is None:
                return self._tensor(term, ops[i]["extents"], cn[i], dense=dense)
            src = self.out_t[prod]
            want = tuple(cn[i][c] for c in term)
            if want == src.counts:
                return src
            key = (prod, want) if share_relayouts else (prod, want, i, k)   # the plan's Cost charges every consuming operand
            if key not in self._relaid:
                dst = self._tensor(term, ops[i]["extents"], cn[i])
                self._relaid[key] = dst
                self.steps.append((f"repartition_{name or prod}_for_{i}", lambda s=src, d=dst: repartition(s.rel, d.rel)))
                self.n_relayouts += 1
            return self._relaid[key]
        self._relaid = {}

        def run(spec, inputs, output):
            return lambda: spec.execute(inputs, output)

        def mm(i, A2, W2, C2, name, addend=None):
            """[rows, j] x [j, k] -> [rows, k] on two-index views; with `addend`, C = A W + addend (fused when the tiling allows)."""
            parts = {"i": A2.splits[0], "j": A2.splits[1], "k": W2.splits[1]}
            if addend is not None and fused:
                sp = Spec("ij,jk,ik->ik", parts, "matmul_add", (), "sum")
                self.steps.append((name + "_add", self._fused_or(sp, [A2, W2, addend], C2,
                                                                 lambda: self._mm_then_add(parts, A2, W2, addend, C2))))
            elif addend is not None:
                self.steps.append((name + "_add", self._mm_then_add(parts, A2, W2, addend, C2)))
            else:
                self.steps.append((name, run(Spec("ij,jk->ik", parts), [A2, W2], C2)))

        # ---- 0: n1 = RMSNorm(x, g1) -------------------------------------------------------------------------------
        self.x = self._tensor("bse", ops[0]["extents"], cn[0])                   # block input, in the tiling operator 0 reads it in
        g1 = operand(0, 1, w["g1"])
        x2, n1 = self.x.rows_view(2), self.out_t[0]
        self.steps.append(("rmsnorm_1", run(Spec("ij,j->ij", {"i": x2.splits[0], "j": x2.splits[1]}, "rmsnorm", (eps,), "none"),
                                           [x2, g1.rel], n1.rows_view(2))))
        # ---- 1-3: q, k, v = n1 W (+ RoPE on q, k) ---------------------------------------------------------------------
        for i, wname, rope in ((1, "wq", True), (2, "wk", True), (3, "wv", False)):
            a = operand(i, 0, name="n1")
            W = operand(i, 1, w[wname].reshape(hidden, n_heads, D))
            A2, W2, out = a.rows_view(2), W.rows_view(1), self.out_t[i]
            if not rope:
                mm(i, A2, W2, out.rows_view(2), f"proj_{wname}")
                continue
            # rows of a two-index view follow the token order only when a row block never mixes sequences with a cut sequence
            natural = cn[i]["s"] == 1 or cn[i]["b"] == batch
            parts = {"i": A2.splits[0], "j": A2.splits[1], "k": W2.splits[1]}
            pre = self._tensor(out.letters, ops[i]["extents"], cn[i])               # before the rotation (unfused chain)
            s_rope = Spec("bshd->bshd", dict(zip("bshd", pre.splits)), "rope", (theta,), "none")

            def unfused(parts=parts, A2=A2, W2=W2, pre=pre, out=out, s_rope=s_rope):
                sp = Spec("ij,jk->ik", parts)
                pv = pre.rows_view(2)
                return lambda: (sp.execute([A2, W2], pv), s_rope.execute([pre.rel], out.rel))
            if fused and natural:
                sp = Spec("ij,jk->ik", parts, "matmul_rope", (theta, seq, D), "sum")
                self.steps.append((f"proj_{wname}_rope", self._fused_or(sp, [A2, W2], out.rows_view(2), unfused)))
            else:
                self.steps.append((f"proj_{wname}_rope", unfused()))
        # ---- 4: attention -------------------------------------------------------------------------------------------
        q, k, v = operand(4, 0, name="q"), operand(4, 1, name="k"), operand(4, 2, name="v")
        att = self.out_t[4]
        c4 = cn[4]
        parts = {"b": ES(batch, c4["b"]), "q": ES(seq, c4["q"]), "h": ES(n_heads, c4["h"]), "d": [0, D], "k": ES(seq, c4["k"])}
        self.steps.append(("attention", run(Spec("bqhd,bkhd,bkhd->bqhd", parts, "attention", (1.0 / math.sqrt(D), 1.0), "online_softmax"),
                                           [q.rel, k.rel, v.rel], att.rel)))
        # ---- 5: h = x + att Wo ----------------------------------------------------------------------------------------
        a = operand(5, 0, name="att")
        Wo = operand(5, 1, w["wo"].reshape(n_heads, D, hidden))
        x5 = self._input_in_tiling(self.x, "bse", ops[5]["extents"], cn[5])
        mm(5, a.rows_view(2), Wo.rows_view(2), self.out_t[5].rows_view(2), "proj_wo", addend=x5.rows_view(2))
        # ---- 6: n2 ----------------------------------------------------------------------------------------------------
        hh = operand(6, 0, name="h")
        g2 = operand(6, 1, w["g2"])
        h2 = hh.rows_view(2)
        self.steps.append(("rmsnorm_2", run(Spec("ij,j->ij", {"i": h2.splits[0], "j": h2.splits[1]}, "rmsnorm", (eps,), "none"),
                                           [h2, g2.rel], self.out_t[6].rows_view(2))))
        # ---- 7-9: silu(n2 W1) * (n2 W3) -------------------------------------------------------------------------------
        a7, a8 = operand(7, 0, name="n2"), operand(8, 0, name="n2")
        W1, W3 = operand(7, 1, w["w1"]), operand(8, 1, w["w3"])
        same = all(cn[7][c] == cn[8][c] == cn[9].get(c, cn[7][c]) for c in "bsf") and cn[7]["e"] == cn[8]["e"]
        done = False
        if fused and same:   # one launch for operators 7, 8 and 9 when they share their tilings
            A2 = a7.rows_view(2)
            parts = {"i": A2.splits[0], "j": A2.splits[1], "k": W1.rel.splits[1]}
            sp = Spec("ij,jk,jk->ik", parts, "swiglu_up", (), "sum")

            def chain():
                s_up = Spec("ij,jk->ik", parts)
                s_silu = Spec("ij,ij->ij", {"i": parts["i"], "j": parts["k"]}, "silu_mul", (), "none")
                o7, o8, o9 = self.out_t[7].rows_view(2), self.out_t[8].rows_view(2), self.out_t[9].rows_view(2)
                return lambda: (s_up.execute([A2, W1.rel], o7), s_up.execute([A2, W3.rel], o8), s_silu.execute([o7, o8], o9))
            self.steps.append(("w13_swiglu", self._fused_or(sp, [A2, W1.rel, W3.rel], self.out_t[9].rows_view(2), chain)))
            done = True
        if not done:
            mm(7, a7.rows_view(2), W1.rel, self.out_t[7].rows_view(2), "proj_w1")
            mm(8, a8.rows_view(2), W3.rel, self.out_t[8].rows_view(2), "proj_w3")
            pa, pb = operand(9, 0, name="a"), operand(9, 1, name="b")
            v9 = self.out_t[9].rows_view(2)
            self.steps.append(("silu_mul", run(Spec("ij,ij->ij", {"i": v9.splits[0], "j": v9.splits[1]}, "silu_mul", (), "none"),
                                              [pa.rows_view(2), pb.rows_view(2)], v9)))
        # ---- 10: out = h + hh W2 ----------------------------------------------------------------------------------------
        a10 = operand(10, 0, name="hh")
        W2 = operand(10, 1, w["w2"])
        h10 = operand(10, 2, name="h")
        mm(10, a10.rows_view(2), W2.rel, self.out_t[10].rows_view(2), "proj_w2", addend=h10.rows_view(2))
        self.out = self.out_t[10]

    # ------------------------------------------------------------------------------------------------------------------
    def _input_in_tiling(self, x: "_Tensor", letters, extents, counts) -> "_Tensor":
        want = tuple(counts[c] for c in letters)
        if want == x.counts:
            return x
        dst = self._tensor(letters, extents, counts)
        self.steps.append(("repartition_x", lambda: repartition(x.rel, dst.rel)))
        self.n_input_relayouts += 1
        return dst

    @staticmethod
    def _mm_then_add(parts, A2, W2, addend, C2):
        tmp = Relation(C2.extents, C2.splits, C2.dtype)
        s_mm = Spec("ij,jk->ik", parts)
        s_add = Spec("ij,ij->ij", {"i": parts["i"], "j": parts["k"]}, "add", (), "none")
        return lambda: (s_mm.execute([A2, W2], tmp), s_add.execute([addend, tmp], C2))

    @staticmethod
    def _fused_or(spec, inputs, output, make_chain):
        """A fused chain; where the library has no fused kernel for the tiling (JA_ERR_UNSUPPORTED, nothing enqueued) the
        chain of separate join-aggs takes its place from then on."""
        state = {"chain": None}

        def call():
            if state["chain"] is None:
                try:
                    spec.execute(inputs, output)
                    return
                except B.JaError as e:
                    if e.status_name != "JA_ERR_UNSUPPORTED":
                        raise
                    state["chain"] = make_chain()
            state["chain"]()
        return call

    def _tensor(self, letters, extents, counts, dense=None):
        return _Tensor(letters, extents, counts, self.dtype, dense)

    def load_input(self, x_dense: torch.Tensor):
        """Pack a dense [batch * seq, hidden] CUDA tensor into the block's input relation (a relayout from one block)."""
        one = from_dense(x_dense.reshape(self.B, self.S, self.hidden), [[0, self.B], [0, self.S], [0, self.hidden]])
        repartition(one, self.x.rel)
        torch.cuda.current_stream().synchronize()

    def forward(self) -> Relation:
        for _, fn in self.steps:
            fn()
        return self.out.rel

    def op_names(self):
        return [n for n, _ in self.steps]

    def flops(self) -> float:
        T, d, f, S = self.T, self.hidden, self.ffn, self.S
        return 2.0 * T * d * d * 4 + 2.0 * T * d * f * 3 + 4.0 * T * S * d / 2


def plan_repartition_charges(ops, counts) -> int:
    """How many (operand, producer) edges of the plan Cost charges a repartition for: the producer's output tiling differs
    from the tiling the consumer's spec reads the operand in (inputs of the computation are never charged)."""
    n = 0
    seen = set()
    for i, op in enumerate(ops):
        ins, _ = _terms(op["einsum"])
        for k, prod in enumerate(op["inputs"]):
            if prod is None:
                continue
            _, pout = _terms(ops[prod]["einsum"])
            have = tuple(counts[prod][c] for c in pout)
            want = tuple(counts[i][c] for c in ins[k])
            if have != want:
                n += 1
                seen.add((prod, want))
    return n, len(seen)
