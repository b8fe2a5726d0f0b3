"""The logical optimizer's plans executed on the GPU (Section 4: Algorithm 1 on the trees that Section 4.5 cuts the block
graph into): `ja_plan_optimize_graph` chooses one join-agg spec per abstract operator of a LLaMA-shaped block, and
`PlannedBlock` turns the interval counts into relations, specs and a `ja_repartition` wherever a producer's output tiling
is not the tiling its consumer's spec reads (sub-cost 1 of Section 4.3). Checked: every intermediate and the output
against the oracle; the number of relayouts executed against the repartition charges in the plan's cost."""
import numpy as np
import pytest
import torch

import paper_2609_03905_b200 as ja
import synth_inputs as si
from oracle import operators, optimizer
from paper_2609_03905_b200.planned_block import PlannedBlock, block_graph, plan_repartition_charges

from gpu_util import TOL, check_status, download, relfro

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


def _oracle_block(x, w, Bt, S, heads):
    w64 = {k: si.to_f64(v) for k, v in w.items()}
    return [operators.llama_block(si.to_f64(x[b * S:(b + 1) * S]), w64, heads) for b in range(Bt)]


def _check_all(blk, refs, Bt, S, hidden, heads):
    D = hidden // heads
    cat = lambda name, shape: np.stack([r[name].reshape(shape) for r in refs])
    for idx, name, shape in ((0, "n1", (S, hidden)), (1, "q", (S, heads, D)), (2, "k", (S, heads, D)), (3, "v", (S, heads, D)),
                             (4, "att", (S, heads, D)), (5, "h", (S, hidden)), (6, "n2", (S, hidden)), (10, "out", (S, hidden))):
        got = download(blk.out_t[idx].rel)
        err = relfro(got, cat(name, shape))
        assert err <= TOL[BF], (name, err)


@pytest.mark.parametrize("p", [8, 64])
@pytest.mark.parametrize("fused", [True, False])
def test_optimizer_plan_on_small_block_every_intermediate(p, fused):
    Bt, S, hidden, heads, ffn = 2, 512, 512, 4, 1408
    ops = block_graph(Bt, S, hidden, heads, ffn)
    cost, plan = ja.ja_plan_optimize_graph(ops, p)
    assert cost == ja.ja_plan_cost(ops, plan) == optimizer.plan_cost(ops, plan)       # the library's plan, costed by the oracle too
    w = si.llama_weights(hidden, ffn, config=5, first_ordinal=21)
    x = si.normal((Bt * S, hidden), 0.0, 1.0, BF, 5, 20)
    blk = PlannedBlock(Bt, S, hidden, heads, ffn, w, plan, fused=fused)
    edges, _ = plan_repartition_charges(ops, plan)
    assert blk.n_relayouts == edges                       # one ja_repartition per repartition charge of the plan's cost
    assert edges > 0                                      # the case does exercise relayouts between operators
    blk.load_input(x.cuda())
    blk.forward()
    check_status()
    _check_all(blk, _oracle_block(x, w, Bt, S, heads), Bt, S, hidden, heads)


def test_hand_plan_with_several_batch_rows_per_block():
    """Batch cut into fewer intervals than it has rows while the sequence is cut too: row blocks of the two-index views are
    (batch interval, sequence interval) pairs, not runs of tokens; RoPE and attention see blocks of two batch rows."""
    Bt, S, hidden, heads, ffn = 4, 256, 512, 4, 1024
    ops = block_graph(Bt, S, hidden, heads, ffn)
    plan = [{"b": 2, "s": 2, "e": 1}, {"b": 2, "s": 2, "e": 2, "h": 1, "d": 1}, {"b": 2, "s": 1, "e": 1, "h": 4, "d": 1},
            {"b": 2, "s": 2, "e": 1, "h": 2, "d": 1}, {"b": 2, "q": 2, "h": 2, "d": 1, "k": 1}, {"b": 2, "s": 2, "h": 1, "d": 1, "e": 2},
            {"b": 2, "s": 2, "e": 2}, {"b": 2, "s": 2, "e": 1, "f": 2}, {"b": 2, "s": 2, "e": 1, "f": 2}, {"b": 2, "s": 2, "f": 2},
            {"b": 4, "s": 1, "f": 2, "e": 1}]
    assert ja.ja_plan_cost(ops, plan) == optimizer.plan_cost(ops, plan)
    w = si.llama_weights(hidden, ffn, config=5, first_ordinal=41)
    x = si.normal((Bt * S, hidden), 0.0, 1.0, BF, 5, 40)
    blk = PlannedBlock(Bt, S, hidden, heads, ffn, w, plan)
    assert blk.n_relayouts == plan_repartition_charges(ops, plan)[0]
    blk.load_input(x.cuda())
    blk.forward()
    check_status()
    _check_all(blk, _oracle_block(x, w, Bt, S, heads), Bt, S, hidden, heads)


@pytest.mark.parametrize("p", [8, 64])
def test_optimizer_plan_on_the_7b_block_sampled_rows(p):
    """Configuration 5 at full size under the optimizer's own plan: output compared with the oracle on sampled token rows
    of one sequence (causal: a prefix is self-contained), and with the hand plan 'seq' on the whole output."""
    from paper_2609_03905_b200.llama_block import LlamaBlock
    Bt, S, hidden, heads, ffn, prefix, seq_id = 8, 2048, 4096, 32, 11008, 512, 5
    ops = block_graph(Bt, S, hidden, heads, ffn)
    cost, plan = ja.ja_plan_optimize_graph(ops, p)
    w = si.llama_weights(hidden, ffn)
    x = si.normal((Bt * S, hidden), 0.0, 1.0, BF, 5, 0)
    blk = PlannedBlock(Bt, S, hidden, heads, ffn, w, plan)
    assert blk.n_relayouts == plan_repartition_charges(ops, plan)[0]
    blk.load_input(x.cuda())
    out = download(blk.forward()).reshape(Bt * S, hidden)
    check_status()
    del blk
    torch.cuda.empty_cache()
    rows = np.unique(np.concatenate([[0, 1, 127, 128, prefix - 1], np.linspace(0, prefix - 1, 6).astype(int)]))
    xs = si.to_f64(x[seq_id * S: seq_id * S + prefix])
    ref = operators.llama_block(xs, {k: si.to_f64(v) for k, v in w.items()}, heads, 1e4, 1e-5, rows=rows)["out"]
    assert relfro(out[seq_id * S + rows], ref) <= TOL[BF]
    hand = LlamaBlock(Bt, S, hidden, heads, ffn, w, plan="seq")
    ja.repartition(ja.from_dense(x.cuda(), [hand.t_sp, hand.io_c]), hand.x)
    assert relfro(out, download(hand.forward())) <= TOL[BF]


def test_greedy_plan_on_small_block():
    """The greedy selector's plan (Section 6, Experiment 3: no repartition sub-cost in the selection) executes like any
    other: one relayout per repartition charge, every intermediate against the oracle; its cost is not below the optimizer's."""
    Bt, S, hidden, heads, ffn = 2, 512, 512, 4, 1408
    ops = block_graph(Bt, S, hidden, heads, ffn)
    cost, plan = ja.ja_plan_select_greedy(ops, 8)
    assert cost == optimizer.plan_cost(ops, plan) and plan == optimizer.greedy(ops, 8)[1]
    assert cost >= ja.ja_plan_optimize_graph(ops, 8)[0]
    w = si.llama_weights(hidden, ffn, config=5, first_ordinal=21)
    x = si.normal((Bt * S, hidden), 0.0, 1.0, BF, 5, 20)
    blk = PlannedBlock(Bt, S, hidden, heads, ffn, w, plan)
    assert blk.n_relayouts == plan_repartition_charges(ops, plan)[0]
    blk.load_input(x.cuda())
    blk.forward()
    check_status()
    _check_all(blk, _oracle_block(x, w, Bt, S, heads), Bt, S, hidden, heads)
