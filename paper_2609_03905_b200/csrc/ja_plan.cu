// Logical optimization (Section 4): one join-agg spec per abstract operator of a computation tree, chosen by the
// dynamic program Opt(Op, T) of Section 4.2 / Algorithm 1 under the communication proxy of Section 4.3. Host code only.
//
// A spec of an operator is the vector of interval counts of its letters (near-equal intervals, Section 3.3); the
// tiling it induces on an operand is the sub-vector of that operand's letters. Sub-costs in closed form:
//   join         sum over operands k of  card(T_k) * prod of the counts of the letters ABSENT from operand k
//                (every cell of operand k is part of one input block per cell of the grid over the absent letters)
//   aggregation  (m - 1) * card(T_out),  m = prod of the counts of the letters absent from the output
//   repartition  card(T_k) when operand k comes from a producer whose output tiling differs from in_k(J)
#include <string.h>

#include <algorithm>
#include <map>
#include <string>
#include <vector>

#include "ja_internal.h"

namespace {

struct Op {
    std::vector<std::string> ins;
    std::string out, letters;
    std::vector<int64_t> extent;      // per letter
    std::vector<int32_t> producers;   // per operand, -1 = input of the computation
    uint32_t fixed = 0;
};
typedef std::vector<int32_t> Counts;   // per letter (a spec) or per index of a tensor (a tiling)

int pos(const std::string& s, char c) {
    size_t p = s.find(c);
    return p == std::string::npos ? -1 : (int)p;
}

ja_status_t parse_op(const ja_plan_node_t& n, int index, Op* op) {
    if (!n.einsum || !n.extents) return ja_fail(JA_ERR_INVALID_ARG, "node %d: einsum / extents missing", index);
    std::string e;
    for (const char* c = n.einsum; *c; ++c)
        if (*c != ' ') e.push_back(*c);
    size_t arrow = e.find("->");
    if (arrow == std::string::npos) return ja_fail(JA_ERR_PARSE, "node %d: einsum '%s' needs '->'", index, n.einsum);
    std::string lhs = e.substr(0, arrow);
    op->out = e.substr(arrow + 2);
    size_t p0 = 0;
    while (true) {
        size_t comma = lhs.find(',', p0);
        op->ins.push_back(lhs.substr(p0, comma == std::string::npos ? std::string::npos : comma - p0));
        if (comma == std::string::npos) break;
        p0 = comma + 1;
    }
    for (const std::string& t : op->ins)
        for (char c : t) {
            if (c < 'a' || c > 'z') return ja_fail(JA_ERR_PARSE, "node %d: bad character '%c'", index, c);
            if (pos(op->letters, c) < 0) op->letters.push_back(c);
        }
    if (op->letters.size() > JA_PLAN_MAX_LETTERS) return ja_fail(JA_ERR_UNSUPPORTED, "node %d: more than %d letters", index, JA_PLAN_MAX_LETTERS);
    for (char c : op->out)
        if (pos(op->letters, c) < 0) return ja_fail(JA_ERR_PARSE, "node %d: output letter '%c' appears in no input", index, c);
    op->extent.assign(n.extents, n.extents + op->letters.size());
    for (int64_t x : op->extent)
        if (x < 1) return ja_fail(JA_ERR_SHAPE, "node %d: extents must be positive", index);
    if (!n.producers) return ja_fail(JA_ERR_INVALID_ARG, "node %d: producers missing", index);
    op->producers.assign(n.producers, n.producers + op->ins.size());
    for (int32_t q : op->producers)
        if (q < -1 || q >= index) return ja_fail(JA_ERR_INVALID_ARG, "node %d: a producer must be an earlier node or -1", index);
    op->fixed = n.fixed_letters;
    return JA_OK;
}

int64_t card(const Op& op, const std::string& term) {
    int64_t n = 1;
    for (char c : term) n *= op.extent[pos(op.letters, c)];
    return n;
}
Counts tiling(const Op& op, const Counts& spec, const std::string& term) {
    Counts t;
    for (char c : term) t.push_back(spec[pos(op.letters, c)]);
    return t;
}
int64_t absent_product(const Op& op, const Counts& spec, const std::string& term) {
    int64_t m = 1;
    for (size_t l = 0; l < op.letters.size(); ++l)
        if (pos(term, op.letters[l]) < 0) m *= spec[l];
    return m;
}
// Cost(J, T_1..T_n); Ts[k] == nullptr for an input of the computation
int64_t cost(const Op& op, const Counts& spec, const std::vector<const Counts*>& Ts) {
    int64_t total = (absent_product(op, spec, op.out) - 1) * card(op, op.out);
    for (size_t k = 0; k < op.ins.size(); ++k) {
        total += card(op, op.ins[k]) * absent_product(op, spec, op.ins[k]);
        if (Ts[k] && *Ts[k] != tiling(op, spec, op.ins[k])) total += card(op, op.ins[k]);
    }
    return total;
}
// specs(Op): interval counts whose product is p, lexicographic over the letters in order of first appearance
void enum_specs(const Op& op, int32_t p, size_t l, Counts* cur, std::vector<Counts>* out) {
    if (l == op.letters.size()) {
        if (p == 1) out->push_back(*cur);
        return;
    }
    if (op.fixed & (1u << l)) {
        cur->push_back(1);
        enum_specs(op, p, l + 1, cur, out);
        cur->pop_back();
        return;
    }
    for (int32_t c = 1; c <= p; ++c) {
        if (p % c || (int64_t)c > op.extent[l]) continue;
        cur->push_back(c);
        enum_specs(op, p / c, l + 1, cur, out);
        cur->pop_back();
    }
}

// What a node can deliver, and at what price: one entry per distinct output tiling the node's specs can produce, holding the
// cheapest total (the node's own Cost plus everything upstream of it inside the tree) of delivering the output in that tiling,
// the spec that achieves it, and -- per operand produced inside the tree -- which entry of the producer's own table it uses.
struct Delivery {
    Counts tiling;                 // of the node's output
    int64_t total;                 // cheapest summed Cost of the subtree that ends in this node, output tiled like this
    Counts spec;                   // the node's spec in that cheapest solution
    std::vector<int> supplier;     // per operand: entry of the producer's table (-1: operand not produced inside the tree)
};
typedef std::vector<Delivery> DeliveryTable;

// allow_sharing = false: every node but the last must be consumed exactly once (a tree, Section 4.2)
ja_status_t parse_all(const ja_plan_node_t* nodes, int32_t n_nodes, bool allow_sharing, std::vector<Op>* ops, std::vector<int>* consumers) {
    if (!nodes || n_nodes < 1) return ja_fail(JA_ERR_INVALID_ARG, "no nodes");
    ops->resize(n_nodes);
    consumers->assign(n_nodes, 0);
    for (int32_t i = 0; i < n_nodes; ++i) {
        ja_status_t st = parse_op(nodes[i], i, &(*ops)[i]);
        if (st != JA_OK) return st;
        const Op& op = (*ops)[i];
        for (size_t k = 0; k < op.ins.size(); ++k) {
            const int32_t q = op.producers[k];
            if (q < 0) continue;
            const Op& pr = (*ops)[q];
            if (pr.out.size() != op.ins[k].size()) return ja_fail(JA_ERR_SHAPE, "node %d operand %zu: rank differs from its producer's output", i, k);
            for (size_t d = 0; d < pr.out.size(); ++d)
                if (pr.extent[pos(pr.letters, pr.out[d])] != op.extent[pos(op.letters, op.ins[k][d])])
                    return ja_fail(JA_ERR_SHAPE, "node %d operand %zu: extent %zu differs from its producer's output", i, k, d);
            if (++(*consumers)[q] > 1 && !allow_sharing)
                return ja_fail(JA_ERR_UNSUPPORTED, "node %d is consumed twice: use ja_plan_optimize_graph, which cuts the graph into trees (Section 4.5)", q);
        }
    }
    if (!allow_sharing)
        for (int32_t i = 0; i + 1 < n_nodes; ++i)
            if ((*consumers)[i] != 1) return ja_fail(JA_ERR_INVALID_ARG, "node %d is not consumed: the last node must be the root of a tree", i);
    return JA_OK;
}

// The dynamic program of Section 4.2 (Algorithm 1) on the tree `members` (ascending = topological) rooted at `root`, stated
// on delivery tables: nodes are visited producers first; for every spec of a node each operand independently picks the
// cheapest entry of its producer's table (entry total + the repartition charge if the entry's tiling is not the one the
// spec reads -- Cost is a sum over operands, so the minimum over all combinations of producer tilings separates), and the
// spec competes for the entry of its own output tiling. The plan is read back from the root's cheapest entry through the
// recorded suppliers.
// Operands from outside the tree: one produced by a node that already has a spec enters with that node's output tiling
// fixed (a mismatch is charged); any other enters like an input of the computation. If `charge_consumers`, the root's entry
// is chosen with the repartition charges of its already-planned consumers added. Fills plan[] for the members.
ja_status_t optimize_tree(const std::vector<Op>& ops, const std::vector<int32_t>& members, int32_t root, int32_t p,
                          bool charge_consumers, std::vector<Counts>* plan, int64_t* tree_cost) {
    std::vector<char> inside(ops.size(), 0);
    for (int32_t i : members) inside[i] = 1;
    std::map<int32_t, DeliveryTable> table;
    for (int32_t i : members) {
        const Op& op = ops[i];
        std::vector<Counts> specs;
        Counts scratch;
        enum_specs(op, p, 0, &scratch, &specs);
        if (specs.empty()) return ja_fail(JA_ERR_TILING, "node %d has no decomposition into %d function specs", i, p);
        const size_t n = op.ins.size();
        enum Source { FREE, IN_TREE, PLANNED_OUTSIDE };
        std::vector<Source> source(n, FREE);
        std::vector<Counts> outside_tiling(n);
        for (size_t k = 0; k < n; ++k) {
            const int32_t q = op.producers[k];
            if (q < 0) continue;
            if (inside[q]) source[k] = IN_TREE;
            else if (!(*plan)[q].empty()) { source[k] = PLANNED_OUTSIDE; outside_tiling[k] = tiling(ops[q], (*plan)[q], ops[q].out); }
        }
        DeliveryTable& mine = table[i];
        for (const Counts& spec : specs) {
            const std::vector<const Counts*> no_producers(n, nullptr);
            Delivery d;
            d.tiling = tiling(op, spec, op.out);
            d.spec = spec;
            d.supplier.assign(n, -1);
            d.total = cost(op, spec, no_producers);          // join + aggregation terms of this node
            for (size_t k = 0; k < n; ++k) {
                const Counts reads = tiling(op, spec, op.ins[k]);
                const int64_t relayout = card(op, op.ins[k]);  // what a mismatch on this operand is charged
                if (source[k] == PLANNED_OUTSIDE) {
                    if (outside_tiling[k] != reads) d.total += relayout;
                } else if (source[k] == IN_TREE) {
                    const DeliveryTable& theirs = table[op.producers[k]];
                    int64_t cheapest = -1;
                    for (size_t e = 0; e < theirs.size(); ++e) {
                        const int64_t v = theirs[e].total + (theirs[e].tiling != reads ? relayout : 0);
                        if (cheapest < 0 || v < cheapest) { cheapest = v; d.supplier[k] = (int)e; }
                    }
                    d.total += cheapest;
                }
            }
            size_t slot = 0;
            while (slot < mine.size() && mine[slot].tiling != d.tiling) ++slot;
            if (slot == mine.size()) mine.push_back(d);
            else if (d.total < mine[slot].total) mine[slot] = d;
        }
    }
    // the root's entry: cheapest once the relayouts its already-planned consumers would need are counted in
    auto consumers_pay = [&](const Counts& T) {
        int64_t c = 0;
        if (!charge_consumers) return c;
        for (size_t j = 0; j < ops.size(); ++j) {
            if ((*plan)[j].empty()) continue;
            for (size_t k = 0; k < ops[j].ins.size(); ++k)
                if (ops[j].producers[k] == root && tiling(ops[j], (*plan)[j], ops[j].ins[k]) != T) c += card(ops[j], ops[j].ins[k]);
        }
        return c;
    };
    const DeliveryTable& top = table[root];
    int chosen = -1;
    int64_t chosen_total = 0;
    for (size_t e = 0; e < top.size(); ++e) {
        const int64_t v = top[e].total + consumers_pay(top[e].tiling);
        if (chosen < 0 || v < chosen_total) { chosen = (int)e; chosen_total = v; }
    }
    if (tree_cost) *tree_cost = top[chosen].total;
    // read the plan back: (node, entry) pairs, following the suppliers
    std::vector<std::pair<int32_t, int>> todo(1, std::make_pair(root, chosen));
    while (!todo.empty()) {
        const int32_t i = todo.back().first;
        const Delivery& d = table[i][todo.back().second];
        todo.pop_back();
        (*plan)[i] = d.spec;
        for (size_t k = 0; k < ops[i].ins.size(); ++k)
            if (d.supplier[k] >= 0) todo.push_back(std::make_pair(ops[i].producers[k], d.supplier[k]));
    }
    return JA_OK;
}

void write_counts(const std::vector<Counts>& plan, int32_t* counts) {
    memset(counts, 0, sizeof(int32_t) * plan.size() * JA_PLAN_MAX_LETTERS);
    for (size_t i = 0; i < plan.size(); ++i)
        for (size_t l = 0; l < plan[i].size(); ++l) counts[i * JA_PLAN_MAX_LETTERS + l] = plan[i][l];
}

int64_t assembled_cost(const std::vector<Op>& ops, const std::vector<Counts>& plan) {
    int64_t total = 0;
    for (size_t i = 0; i < ops.size(); ++i) {
        std::vector<Counts> outs(ops[i].ins.size());
        std::vector<const Counts*> Ts(ops[i].ins.size(), nullptr);
        for (size_t k = 0; k < ops[i].ins.size(); ++k)
            if (ops[i].producers[k] >= 0) {
                outs[k] = tiling(ops[ops[i].producers[k]], plan[ops[i].producers[k]], ops[ops[i].producers[k]].out);
                Ts[k] = &outs[k];
            }
        total += cost(ops[i], plan[i], Ts);
    }
    return total;
}

}  // namespace

extern "C" ja_status_t ja_plan_optimize(const ja_plan_node_t* nodes, int32_t n_nodes, int32_t p, int32_t* counts, int64_t* total_cost) {
    if (p < 1 || !counts) return ja_fail(JA_ERR_INVALID_ARG, "p must be positive and counts non-NULL");
    std::vector<Op> ops;
    std::vector<int> consumers;
    ja_status_t st = parse_all(nodes, n_nodes, false, &ops, &consumers);
    if (st != JA_OK) return st;
    std::vector<int32_t> members(n_nodes);
    for (int32_t i = 0; i < n_nodes; ++i) members[i] = i;
    std::vector<Counts> plan(n_nodes);
    if ((st = optimize_tree(ops, members, n_nodes - 1, p, false, &plan, total_cost)) != JA_OK) return st;
    write_counts(plan, counts);
    return JA_OK;
}

extern "C" ja_status_t ja_plan_optimize_graph(const ja_plan_node_t* nodes, int32_t n_nodes, int32_t p, int32_t* counts, int64_t* total_cost) {
    if (p < 1 || !counts) return ja_fail(JA_ERR_INVALID_ARG, "p must be positive and counts non-NULL");
    std::vector<Op> ops;
    std::vector<int> consumers;
    ja_status_t st = parse_all(nodes, n_nodes, true, &ops, &consumers);
    if (st != JA_OK) return st;
    // cut at every edge out of a multiply consumed tensor: roots are the nodes not consumed exactly once
    std::vector<std::pair<int32_t, std::vector<int32_t>>> trees;
    for (int32_t root = 0; root < n_nodes; ++root) {
        if (consumers[root] == 1) continue;
        std::vector<int32_t> members, stack(1, root);
        while (!stack.empty()) {
            const int32_t i = stack.back();
            stack.pop_back();
            members.push_back(i);
            for (int32_t q : ops[i].producers)
                if (q >= 0 && consumers[q] == 1) stack.push_back(q);
        }
        std::sort(members.begin(), members.end());
        trees.push_back({root, members});
    }
    std::stable_sort(trees.begin(), trees.end(), [](const std::pair<int32_t, std::vector<int32_t>>& a, const std::pair<int32_t, std::vector<int32_t>>& b) {
        return a.second.size() != b.second.size() ? a.second.size() > b.second.size() : a.first < b.first;
    });
    std::vector<Counts> plan(n_nodes);
    for (const auto& t : trees)
        if ((st = optimize_tree(ops, t.second, t.first, p, true, &plan, nullptr)) != JA_OK) return st;
    write_counts(plan, counts);
    if (total_cost) *total_cost = assembled_cost(ops, plan);
    return JA_OK;
}

// The greedy selector of the paper's plan-selection experiment (Section 6, Experiment 3): the same program with the
// repartition sub-cost removed. That sub-cost is the only one that depends on the producers' tilings, so the recurrence falls
// apart and every operator takes, on its own, the spec with the least join + aggregation cost (the first such spec in the
// enumeration order of specs(Op)). The cost reported is the plan's full Cost, repartition charges included.
extern "C" ja_status_t ja_plan_select_greedy(const ja_plan_node_t* nodes, int32_t n_nodes, int32_t p, int32_t* counts, int64_t* total_cost) {
    if (p < 1 || !counts) return ja_fail(JA_ERR_INVALID_ARG, "p must be positive and counts non-NULL");
    std::vector<Op> ops;
    std::vector<int> consumers;
    ja_status_t st = parse_all(nodes, n_nodes, true, &ops, &consumers);
    if (st != JA_OK) return st;
    std::vector<Counts> plan(n_nodes);
    for (int32_t i = 0; i < n_nodes; ++i) {
        std::vector<Counts> cand;
        Counts cur;
        enum_specs(ops[i], p, 0, &cur, &cand);
        if (cand.empty()) return ja_fail(JA_ERR_TILING, "node %d has no spec with %d function specs", i, p);
        const std::vector<const Counts*> no_producers(ops[i].ins.size(), nullptr);
        int64_t best = -1;
        for (const Counts& J : cand) {
            const int64_t c = cost(ops[i], J, no_producers);
            if (best < 0 || c < best) { best = c; plan[i] = J; }
        }
    }
    write_counts(plan, counts);
    if (total_cost) *total_cost = assembled_cost(ops, plan);
    return JA_OK;
}

extern "C" ja_status_t ja_plan_cost(const ja_plan_node_t* nodes, int32_t n_nodes, const int32_t* counts, int64_t* total_cost) {
    if (!counts || !total_cost) return ja_fail(JA_ERR_INVALID_ARG, "counts / total_cost is NULL");
    std::vector<Op> ops;
    std::vector<int> consumers;
    ja_status_t st = parse_all(nodes, n_nodes, true, &ops, &consumers);
    if (st != JA_OK) return st;
    std::vector<Counts> plan(n_nodes);
    for (int32_t i = 0; i < n_nodes; ++i) {
        const Op& op = ops[i];
        for (size_t l = 0; l < op.letters.size(); ++l) {
            const int32_t c = counts[(size_t)i * JA_PLAN_MAX_LETTERS + l];
            if (c < 1 || c > op.extent[l]) return ja_fail(JA_ERR_TILING, "node %d letter '%c': %d intervals", i, op.letters[l], c);
            plan[i].push_back(c);
        }
    }
    *total_cost = assembled_cost(ops, plan);
    return JA_OK;
}
