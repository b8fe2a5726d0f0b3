"""A LLaMA-shaped transformer block forward as a chain of join-aggs: nothing here computes -- every step is
one ja_execute or ja_repartition call on relations allocated up front.

    n1 = RMSNorm(x, g1);  q,k,v = n1 Wq, n1 Wk, n1 Wv;  q,k <- RoPE;  att = CausalAttention(q,k,v)
    h  = x + att Wo;      n2 = RMSNorm(h, g2);  out = h + (silu(n2 W1) * (n2 W3)) W2

Two decompositions (the block's input and output relations are tiled identically in both: 128-token row
blocks x 8 column blocks):

  "seq"   sequence-blocked: every [tokens, hidden] relation keeps 128 x (hidden/8) blocks; q, k, v are
          re-tiled to one head per block before attention and the attention output is re-tiled back
          (the one-GPU image of sequence-parallel outside / head-parallel inside attention).
  "head"  head-blocked: x is re-tiled once to 128 x 128 blocks (one head per column block); all projections
          contract over 32 (64) head-sized blocks and emit head-sized blocks, so attention needs no
          relayout; the block output is re-tiled back at the end.
  "mixed" sequence-blocked everywhere, attention included: its spec cuts the head index into as many intervals as the
          activations have column blocks (several heads per block), so q, k, v are consumed in the tiling their
          projections emit and the attention output in the tiling the output projection contracts over: no relayout
          anywhere inside the block.
"""
from __future__ import annotations

import math

import torch

from . import binding as B
from .relations import Relation, Spec, equal_splits as ES, from_dense, repartition


class LlamaBlock:
    def __init__(self, batch: int, seq: int, hidden: int, n_heads: int, ffn: int, weights: dict, plan: str = "seq",
                 theta: float = 1e4, eps: float = 1e-5, token_block: int = 128, col_blocks: int = 8,
                 ffn_blocks: int | None = None, fused: bool = True, n_kv_heads: int | None = None,
                 dtype: torch.dtype = torch.bfloat16):
        assert plan in ("seq", "head", "mixed")
        self.fused = fused
        assert hidden % n_heads == 0 and hidden // n_heads == 128, "attention kernel needs head dimension 128"
        assert seq % token_block == 0
        self.plan, self.B, self.S, self.hidden, self.H, self.ffn = plan, batch, seq, hidden, n_heads, ffn
        n_kv = n_heads if n_kv_heads is None else n_kv_heads       # grouped-query attention (Example 3.10) when smaller
        assert n_heads % n_kv == 0
        self.n_kv, self.kv_hidden = n_kv, n_kv * (hidden // n_heads)
        kv_hidden = self.kv_hidden
        T = batch * seq
        self.T = T
        assert dtype in (torch.bfloat16, torch.float16), "the block's relations are bf16 (the benchmark configurations) or f16 (the paper's precision)"
        bf = self.dtype = dtype                          # cell type of every relation of the block
        D = hidden // n_heads
        t_sp = ES(T, T // token_block)
        io_c = ES(hidden, col_blocks)                    # column tiling of the block's input / output
        head_c = ES(hidden, n_kv)                        # one key/value head's group of query heads per column block
        kvhead_c = ES(kv_hidden, n_kv)                   # one key/value head per column block
        act_c = head_c if plan == "head" else io_c       # column tiling of the plan's [T, hidden] activations
        # the FFN index is cut into 256-wide blocks when it divides evenly (11008 = 43 x 256, 22016 = 86 x 256): every
        # output tile of the up-projections is then a whole block, with no ragged tail tile per block
        if ffn_blocks is None:
            ffn_blocks = ffn // 256 if ffn % 256 == 0 else col_blocks
        ffn_c = ES(ffn, ffn_blocks)
        self.t_sp, self.io_c, self.head_c, self.act_c, self.ffn_c = t_sp, io_c, head_c, act_c, ffn_c
        # tilings q and k, v are produced in: column blocks hold whole heads, so the narrower key/value relations may get
        # fewer blocks; plan "mixed" feeds them to attention as they are, so there q is cut like k, v (grouped heads)
        n_kvb = min(col_blocks, n_kv)
        qkv_c = {"seq": io_c, "head": head_c, "mixed": ES(hidden, n_kvb)}[plan]
        kv_c = kvhead_c if plan == "head" else ES(kv_hidden, n_kvb)
        att_c = head_c if plan != "mixed" else qkv_c     # tiling attention reads q from and writes its output in
        kvatt_c = kvhead_c if plan != "mixed" else kv_c

        def act(cols=act_c):
            return Relation([T, hidden], [t_sp, cols], bf)

        def kv(cols=kv_c):
            return Relation([T, kv_hidden], [t_sp, cols], bf)

        # ---- relations -------------------------------------------------------------------------------
        self.x = Relation([T, hidden], [t_sp, io_c], bf)                 # block input (filled by the caller)
        self.out = Relation([T, hidden], [t_sp, io_c], bf)               # block output
        self.x_p = act() if plan == "head" else self.x                   # input in the plan's tiling
        self.n1, self.h, self.n2, self.o, self.y = act(), act(), act(), act(), act()
        self.q, self.k, self.v = act(qkv_c), kv(), kv()
        self.q_r, self.k_r = act(qkv_c), kv()                            # after RoPE
        if plan == "seq":
            self.q_h, self.k_h, self.v_h, self.att_h = act(head_c), kv(kvhead_c), kv(kvhead_c), act(head_c)
            self.att = act()
        else:
            self.q_h, self.k_h, self.v_h = self.q_r, self.k_r, self.v
            self.att_h = self.att = act(att_c)
        self.out_p = act() if plan == "head" else self.out
        self.a = Relation([T, ffn], [t_sp, ffn_c], bf)
        self.b = Relation([T, ffn], [t_sp, ffn_c], bf)
        self.hh = Relation([T, ffn], [t_sp, ffn_c], bf)
        # weights [in, out]: rows tiled like the activation they contract with, columns like the result
        w = {n: weights[n].to("cuda", bf) for n in weights}
        self.wq = from_dense(w["wq"], [act_c, qkv_c])
        self.wk, self.wv = (from_dense(w[n], [act_c, kv_c]) for n in ("wk", "wv"))
        self.wo = from_dense(w["wo"], [io_c if plan == "seq" else att_c, act_c])
        self.w1, self.w3 = from_dense(w["w1"], [act_c, ffn_c]), from_dense(w["w3"], [act_c, ffn_c])
        self.w2 = from_dense(w["w2"], [ffn_c, act_c])
        self.g1, self.g2 = from_dense(w["g1"], [act_c]), from_dense(w["g2"], [act_c])

        # 4-D views "bshd" over the same payloads (the block layout of [T, hidden] with 128-token row blocks
        # and whole-head column blocks IS the layout of [b, s, h, d] with blocks [1, 128, heads/block, 128])
        b_sp, s_sp = ES(batch, batch), ES(seq, seq // token_block)

        def v4(rel: Relation, cols, heads=n_heads):
            hb = ES(heads, len(cols) - 1)
            return rel.view_as([batch, seq, heads, D], [b_sp, s_sp, hb, [0, D]])

        self.q4, self.k4 = v4(self.q, qkv_c), v4(self.k, kv_c, n_kv)
        self.q4r, self.k4r = v4(self.q_r, qkv_c), v4(self.k_r, kv_c, n_kv)
        self.qa, self.oa = v4(self.q_h, att_c), v4(self.att_h, att_c)
        self.ka, self.va = v4(self.k_h, kvatt_c, n_kv), v4(self.v_h, kvatt_c, n_kv)

        # ---- specs -------------------------------------------------------------------------------------
        def mm(jc, kc):
            return Spec("ij,jk->ik", {"i": t_sp, "j": jc, "k": kc}, "mul", (), "sum")

        self.s_norm = Spec("ij,j->ij", {"i": t_sp, "j": act_c}, "rmsnorm", (eps,), "none")
        self.s_qkv = mm(act_c, qkv_c)
        self.s_kv = mm(act_c, kv_c)
        self.s_rope = Spec("bshd->bshd", {"b": b_sp, "s": s_sp, "h": ES(n_heads, len(qkv_c) - 1), "d": [0, D]}, "rope",
                           (theta,), "none")
        self.s_rope_k = Spec("bshd->bshd", {"b": b_sp, "s": s_sp, "h": ES(n_kv, len(kv_c) - 1), "d": [0, D]}, "rope",
                             (theta,), "none")
        n_hb = len(att_c) - 1                             # intervals of the head index in the attention spec
        if n_kv == n_heads:
            self.s_attn = Spec("bqhd,bkhd,bkhd->bqhd", {"b": b_sp, "q": s_sp, "h": ES(n_heads, n_hb), "d": [0, D], "k": s_sp},
                               "attention", (1.0 / math.sqrt(D), 1.0), "online_softmax")
        else:   # query heads inherit their split from the key/value heads: intervals of n_heads / n_kv heads per key/value head
            self.s_attn = Spec("bqhd,bkgd,bkgd->bqhd", {"b": b_sp, "q": s_sp, "h": ES(n_heads, n_hb), "d": [0, D], "k": s_sp,
                                                         "g": ES(n_kv, n_hb)}, "attention", (1.0 / math.sqrt(D), 1.0), "online_softmax")
        self.s_wo = mm(io_c if plan == "seq" else att_c, act_c)
        self.s_add = Spec("ij,ij->ij", {"i": t_sp, "j": act_c}, "add", (), "none")
        self.s_up = mm(act_c, ffn_c)
        self.s_silu = Spec("ij,ij->ij", {"i": t_sp, "j": ffn_c}, "silu_mul", (), "none")
        self.s_down = mm(ffn_c, act_c)
        self.n_relayouts = {"seq": 4, "head": 2, "mixed": 0}[plan]
        # fused chains: the projection's accumulator goes through RoPE / the residual ADD / SILU_MUL before its store
        # (a fused form that the tiling cannot run -- JA_ERR_UNSUPPORTED -- falls back to its chain, once and for all)
        self.fuse_rope = self.fuse_add = self.fuse_swiglu = fused
        if fused:
            self.s_qk_rope = Spec("ij,jk->ik", {"i": t_sp, "j": act_c, "k": qkv_c}, "matmul_rope", (theta, seq, D), "sum")
            self.s_k_rope = Spec("ij,jk->ik", {"i": t_sp, "j": act_c, "k": kv_c}, "matmul_rope", (theta, seq, D), "sum")
            self.s_wo_add = Spec("ij,jk,ik->ik", {"i": t_sp, "j": io_c if plan == "seq" else att_c, "k": act_c}, "matmul_add", (), "sum")
            self.s_up_swiglu = Spec("ij,jk,jk->ik", {"i": t_sp, "j": act_c, "k": ffn_c}, "swiglu_up", (), "sum")
            self.s_down_add = Spec("ij,jk,ik->ik", {"i": t_sp, "j": ffn_c, "k": act_c}, "matmul_add", (), "sum")

    # flop count of one forward (dense contractions only; causal attention counted at half the square)
    def flops(self) -> float:
        T, d, f, S = self.T, self.hidden, self.ffn, self.S
        return 2.0 * T * d * (2 * d + 2 * self.kv_hidden) + 2.0 * T * d * f * 3 + 4.0 * T * S * d / 2

    @staticmethod
    def _fused(spec: Spec, inputs, output: Relation, stream) -> bool:
        """Run a fused chain; False if libja has no fused kernel for this tiling (nothing was enqueued)."""
        try:
            spec.execute(inputs, output, stream)
            return True
        except B.JaError as e:
            if e.status_name != "JA_ERR_UNSUPPORTED":
                raise
            return False

    def op_names(self):
        """Names of the libja calls of one forward(), in order (for per-op timing)."""
        n = ["repartition_x"] if self.plan == "head" else []
        n += ["rmsnorm_1"]
        n += ["q_proj_rope", "k_proj_rope", "v_proj"] if self.fuse_rope else ["q_proj", "k_proj", "v_proj", "rope_q", "rope_k"]
        n += ["repartition_q", "repartition_k", "repartition_v"] if self.plan == "seq" else []
        n += ["attention"]
        n += ["repartition_att"] if self.plan == "seq" else []
        n += ["o_proj_add"] if self.fuse_add else ["o_proj", "residual_1"]
        n += ["rmsnorm_2"]
        n += ["w13_swiglu"] if self.fuse_swiglu else ["w1_proj", "w3_proj", "silu_mul"]
        n += ["w2_proj_add"] if self.fuse_add else ["w2_proj", "residual_2"]
        n += ["repartition_out"] if self.plan == "head" else []
        return n

    def capture(self):
        """The whole chain as one CUDA graph (the paper builds one graph per plan): returns a torch.cuda.CUDAGraph whose
        replay() re-runs forward() on the relations of this block. Call forward() once before, so that every plan and
        device table the library caches exists (creating them allocates, which a capture does not allow)."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.forward()
        return g

    def forward(self, stream: int | None = None) -> Relation:
        """Enqueue the whole chain on the current stream; returns the output relation (tiled like x)."""
        p = self.plan
        if p == "head":
            repartition(self.x, self.x_p, stream)
        self.s_norm.execute([self.x_p, self.g1], self.n1, stream)
        if self.fuse_rope and not self._fused(self.s_qk_rope, [self.n1, self.wq], self.q_r, stream):
            self.fuse_rope = False
        if self.fuse_rope:
            self.s_k_rope.execute([self.n1, self.wk], self.k_r, stream)
            self.s_kv.execute([self.n1, self.wv], self.v, stream)
        else:
            self.s_qkv.execute([self.n1, self.wq], self.q, stream)
            self.s_kv.execute([self.n1, self.wk], self.k, stream)
            self.s_kv.execute([self.n1, self.wv], self.v, stream)
            self.s_rope.execute([self.q4], self.q4r, stream)
            self.s_rope_k.execute([self.k4], self.k4r, stream)
        if p == "seq":
            repartition(self.q_r, self.q_h, stream)
            repartition(self.k_r, self.k_h, stream)
            repartition(self.v, self.v_h, stream)
        self.s_attn.execute([self.qa, self.ka, self.va], self.oa, stream)
        if p == "seq":
            repartition(self.att_h, self.att, stream)
        if self.fuse_add and not self._fused(self.s_wo_add, [self.att, self.wo, self.x_p], self.h, stream):
            self.fuse_add = False
        if not self.fuse_add:
            self.s_wo.execute([self.att, self.wo], self.o, stream)
            self.s_add.execute([self.x_p, self.o], self.h, stream)
        self.s_norm.execute([self.h, self.g2], self.n2, stream)
        if self.fuse_swiglu and not self._fused(self.s_up_swiglu, [self.n2, self.w1, self.w3], self.hh, stream):
            self.fuse_swiglu = False
        if not self.fuse_swiglu:
            self.s_up.execute([self.n2, self.w1], self.a, stream)
            self.s_up.execute([self.n2, self.w3], self.b, stream)
            self.s_silu.execute([self.a, self.b], self.hh, stream)
        if self.fuse_add:
            self.s_down_add.execute([self.hh, self.w2, self.h], self.out_p, stream)
        else:
            self.s_down.execute([self.hh, self.w2], self.y, stream)
            self.s_add.execute([self.h, self.y], self.out_p, stream)
        if p == "head":
            repartition(self.out_p, self.out, stream)
        return self.out
