"""TEST INFRASTRUCTURE ONLY -- exchange programs (paper Section 5, "Physical Optimization").

Written from Section 5.2 (the ExProg language: state, GPUS / PARTITIONS / IN / OUT, actions, the three rules, the cost
model of the hardware simulator), Section 5.3 (overlay atoms, the generated preamble) and Section 5.4 (Definition
"Closure; validity", Insert / Delete, the four families of rewriting rules).  Plain Python over frozensets; nothing here
is shared with the library's C++ implementation.

Text form accepted (a reading of the printed examples):
    GPUS: 0, 1, 2, 3                          optional; default = the sites named anywhere in the program
    PARTITIONS: G1 {size 2} G2 {2, 3}         by size (membership chosen later) or by explicit members
    IN:  A @ 0 (size: 1.0 GB); B @ 1          ';' or a line break between items, sizes default to 1 GB
    OUT: A+B @ 0, 1; C @ G1
    <blank line>
    A @ 0 -> 1;  B @ 1 -> 0;  A+B @ 0, 1      the body: a SET of actions "aggregate @ source(s) [-> destinations]"
An action with an arrow has one source site; without an arrow the source may be a list of sites or a partition name
(one local aggregation per site).

Readings where the paper is silent:
  * all atoms of one aggregate are copies of one tensor block, so an aggregate has the size of any of its atoms;
  * a local aggregation of m >= 2 materialised parts reads m and writes 1 block of that size at the site's HBM bandwidth;
    an aggregate that is already materialised at the source costs nothing (m = 1);
  * an action starts when some set of aggregates materialised at its source partitions its aggregate, and uses the
    partition with the fewest parts available at that moment; its transfer starts when its aggregation ends;
  * concurrent work shares a resource equally: aggregations at one site share its HBM bandwidth; on an NVSwitch fabric a
    flow gets min(egress of its source / flows leaving it, ingress of its destination / flows entering it), a multicast
    to k sites being k flows; on the cube mesh flows on one directed link share it, and all flows between unlinked pairs
    share the PCIe bridge;
  * the cube mesh (the paper names only the four 50 GB/s pillars and says that pairs inside a CPU socket have single links): sites {0,1,2,3} and
    {4,5,6,7} are fully connected by 25 GB/s links, i <-> i+4 are 50 GB/s, every other pair goes over PCIe;
  * the completion time is the time at which the last action of the program finishes.
"""
from __future__ import annotations

import itertools
import math
import re
from dataclasses import dataclass, field


# ------------------------------------------------------------------------------------------------- data model
@dataclass
class Program:
    gpus: list                                   # valid sites
    partitions: dict = field(default_factory=dict)   # name -> {"size": n, "members": tuple | None}
    atoms: dict = field(default_factory=dict)        # name -> (site, size in GB), in declaration order
    out: list = field(default_factory=list)          # (frozenset of atom names, ("sites", tuple) | ("part", name))
    actions: list = field(default_factory=list)      # (frozenset, ("sites", tuple) | ("part", name), tuple of destination sites)

    def copy(self):
        return Program(list(self.gpus), {k: dict(v) for k, v in self.partitions.items()}, dict(self.atoms),
                       list(self.out), list(self.actions))


_KEYWORDS = ("GPUS", "PARTITIONS", "IN", "OUT")


def _items(text):
    return [t.strip() for t in re.split(r"[;\n]", text) if t.strip()]


def _sites(text):
    return tuple(int(t) for t in (u.strip() for u in text.split(",")) if t != "")


def _target(text, partitions):
    text = text.strip()
    if text in partitions:
        return ("part", text)
    return ("sites", _sites(text))


def parse(text: str) -> Program:
    """Section 5.2: preamble (GPUS, PARTITIONS, IN, OUT) and body."""
    m = re.search(r"\bOUT\s*:", text)
    if not m:
        raise ValueError("no OUT declaration")
    blank = re.search(r"\n[ \t]*\n", text[m.end():])
    pre = text if not blank else text[:m.end() + blank.start()]
    body = "" if not blank else text[m.end() + blank.end():]
    marks = sorted((mm.start(), mm.end(), mm.group(1)) for mm in re.finditer(r"\b(GPUS|PARTITIONS|IN|OUT)\s*:", pre))
    sect = {}
    for i, (a, b, kw) in enumerate(marks):
        sect[kw] = pre[b:marks[i + 1][0] if i + 1 < len(marks) else len(pre)]
    prog = Program([])
    for name, inner in re.findall(r"(\w+)\s*\{([^}]*)\}", sect.get("PARTITIONS", "")):
        inner = inner.strip()
        ms = re.fullmatch(r"size\s+(\d+)", inner)
        if ms:
            prog.partitions[name] = {"size": int(ms.group(1)), "members": None}
        else:
            mem = _sites(inner)
            prog.partitions[name] = {"size": len(mem), "members": mem}
    for it in _items(sect["IN"]):
        mi = re.fullmatch(r"(\w+)\s*@\s*(\d+)\s*(?:\(\s*size\s*:\s*([0-9.eE+-]+)\s*GB\s*\))?", it)
        if not mi:
            raise ValueError("bad IN item: " + it)
        if mi.group(1) in prog.atoms:
            raise ValueError("atom declared twice: " + mi.group(1))
        prog.atoms[mi.group(1)] = (int(mi.group(2)), float(mi.group(3)) if mi.group(3) else 1.0)
    if not prog.atoms:
        raise ValueError("IN declares no atom")

    def aggregate(t):
        names = [n.strip() for n in t.split("+")]
        if len(set(names)) != len(names) or any(n not in prog.atoms for n in names):
            raise ValueError("bad aggregate: " + t)
        return frozenset(names)

    for it in _items(sect["OUT"]):
        agg, where = it.split("@")
        prog.out.append((aggregate(agg), _target(where, prog.partitions)))
    for it in _items(body):
        left, _, right = it.partition("->")
        agg, where = left.split("@")
        src = _target(where, prog.partitions)
        dests = _sites(right) if right.strip() else ()
        if dests and (src[0] != "sites" or len(src[1]) != 1):
            raise ValueError("an action with an arrow has one source site: " + it)
        act = (aggregate(agg), src, dests)
        if act not in prog.actions:               # a program is a set
            prog.actions.append(act)
    if "GPUS" in sect:
        prog.gpus = list(_sites(sect["GPUS"]))
    else:
        seen = {s for s, _ in prog.atoms.values()}
        for _, tg in prog.out:
            seen |= set(tg[1]) if tg[0] == "sites" else set()
        for _, src, d in prog.actions:
            seen |= set(d) | (set(src[1]) if src[0] == "sites" else set())
        for p in prog.partitions.values():
            seen |= set(p["members"] or ())
        prog.gpus = sorted(seen)
    _check_static(prog)
    return prog


def _check_static(prog: Program):
    g = set(prog.gpus)
    fixed = [s for p in prog.partitions.values() if p["members"] is not None for s in p["members"]]
    if len(fixed) != len(set(fixed)) or not set(fixed) <= g:
        raise ValueError("partitions overlap or name an undeclared site")
    if prog.partitions and sum(p["size"] for p in prog.partitions.values()) != len(g):
        raise ValueError("partitions must cover the declared GPUs")       # Section 5.2: disjoint and covering
    for s, _ in prog.atoms.values():
        if s not in g:
            raise ValueError("atom at an undeclared site")
    for agg, tg in prog.out:
        if len({prog.atoms[a][1] for a in agg}) != 1:
            raise ValueError("atoms of one aggregate differ in size")
        if tg[0] == "sites" and not set(tg[1]) <= g:
            raise ValueError("OUT names an undeclared site")
    for agg, src, d in prog.actions:
        if len({prog.atoms[a][1] for a in agg}) != 1:
            raise ValueError("atoms of one aggregate differ in size")
        if not set(d) <= g or (src[0] == "sites" and not set(src[1]) <= g):
            raise ValueError("an action names an undeclared site")


def merge(a: Program, b: Program, prefix_a: str, prefix_b: str) -> Program:
    """One program out of two over the same GPUS and PARTITIONS: the exchanges of two operands of one operator, which share
    the placement of its function specs and run at the same time (Section 5.1 compiles one program per operator)."""
    if a.gpus != b.gpus or a.partitions != b.partitions:
        raise ValueError("the two preambles disagree")
    q = Program(list(a.gpus), {k: dict(v) for k, v in a.partitions.items()})
    for prog, pre in ((a, prefix_a), (b, prefix_b)):
        for n, v in prog.atoms.items():
            if pre + n in q.atoms:
                raise ValueError("atom names clash")
            q.atoms[pre + n] = v
        q.out += [(frozenset(pre + n for n in x), t) for x, t in prog.out]
        for x, src, d in prog.actions:
            act = (frozenset(pre + n for n in x), src, d)
            if act not in q.actions:
                q.actions.append(act)
    _check_static(q)
    return q


def _name_order(prog):
    return {a: i for i, a in enumerate(prog.atoms)}


def format_program(prog: Program) -> str:
    order = _name_order(prog)

    def agg(x):
        return "+".join(sorted(x, key=order.get))

    def tgt(t):
        return t[1] if t[0] == "part" else ", ".join(str(s) for s in t[1])

    lines = ["GPUS: " + ", ".join(str(s) for s in prog.gpus)]
    if prog.partitions:
        lines.append("PARTITIONS: " + " ".join(
            "%s {%s}" % (n, "size %d" % p["size"] if p["members"] is None else ", ".join(str(s) for s in p["members"]))
            for n, p in prog.partitions.items()))
    lines.append("IN: " + "; ".join(
        "%s @ %d" % (a, s) + ("" if gb == 1.0 else " (size: %r GB)" % gb) for a, (s, gb) in prog.atoms.items()))
    lines.append("OUT: " + "; ".join("%s @ %s" % (agg(x), tgt(t)) for x, t in prog.out))
    lines.append("")
    for x, src, d in prog.actions:
        lines.append("%s @ %s" % (agg(x), tgt(src)) + (" -> " + ", ".join(str(s) for s in d) if d else ""))
    return "\n".join(lines) + "\n"


# ------------------------------------------------------------------------------------- memberships of partitions
def memberships(prog: Program):
    """Every choice of members for the partitions declared by size alone (Section 5.2: disjoint, covering the GPUs)."""
    names = [n for n, p in prog.partitions.items() if p["members"] is None]
    taken = {s for p in prog.partitions.values() if p["members"] is not None for s in p["members"]}
    free = [s for s in prog.gpus if s not in taken]

    def rec(i, rest):
        if i == len(names):
            yield {}
            return
        for mem in itertools.combinations(rest, prog.partitions[names[i]]["size"]):
            left = [s for s in rest if s not in mem]
            for tail in rec(i + 1, left):
                yield {names[i]: mem, **tail}

    yield from rec(0, free)


def bind(prog: Program, membership: dict) -> Program:
    """The program with the given members written into its size-declared partitions."""
    q = prog.copy()
    for n, mem in membership.items():
        if q.partitions[n]["members"] is None and len(mem) != q.partitions[n]["size"]:
            raise ValueError("wrong size for partition " + n)
        q.partitions[n]["members"] = tuple(sorted(mem))
    _check_static(q)
    return q


def _resolve(prog, target):
    if target[0] == "sites":
        return tuple(target[1])
    mem = prog.partitions[target[1]]["members"]
    if mem is None:
        raise ValueError("partition %s has no members yet" % target[1])
    return tuple(mem)


def expanded(prog: Program):
    """The actions with one source site each: (aggregate, site, destinations), as a list without duplicates."""
    res = []
    for x, src, d in prog.actions:
        for s in _resolve(prog, src):
            a = (x, s, tuple(d))
            if a not in res:
                res.append(a)
    return res


def requirements(prog: Program):
    return [(x, s) for x, t in prog.out for s in _resolve(prog, t)]


# ------------------------------------------------------------------------- Definition "Closure; validity" (Section 5.4)
def exact_cover(x: frozenset, available, order=None):
    """A partition of x into members of `available` with the fewest parts (None if there is none).  With `order` (atom ->
    position) the search branches on the first uncovered atom in that order, so the parts come out by their first atoms."""
    cands = [y for y in available if y and y <= x]
    best = [None]

    def rec(rest, parts):
        if best[0] is not None and len(parts) >= len(best[0]):
            return
        if not rest:
            best[0] = list(parts)
            return
        pivot = min(rest) if order is None else min(rest, key=order.get)
        for y in cands:
            if pivot in y and y <= rest:
                parts.append(y)
                rec(rest - y, parts)
                parts.pop()

    rec(x, [])
    return best[0]


def closure(prog: Program):
    """S*(P): the least state containing the initial state and closed under firing the enabled actions of P."""
    state = {(frozenset([a]), s) for a, (s, _) in prog.atoms.items()}
    acts = expanded(prog)
    changed = True
    while changed:
        changed = False
        for x, s, d in acts:
            here = [y for y, t in state if t == s]
            if exact_cover(x, here) is None:
                continue
            new = {(x, s)} | {(x, t) for t in d}
            if not new <= state:
                state |= new
                changed = True
    return state


def well_formed(prog: Program) -> bool:
    state = closure(prog)
    return all(exact_cover(x, [y for y, t in state if t == s]) is not None for x, s, _ in expanded(prog))


def valid_bound(prog: Program) -> bool:
    """Validity with every partition's membership fixed."""
    state = closure(prog)
    if not all(exact_cover(x, [y for y, t in state if t == s]) is not None for x, s, _ in expanded(prog)):
        return False
    return all((x, s) in state for x, s in requirements(prog))


def valid(prog: Program) -> bool:
    """Valid if some choice of membership for the size-declared partitions makes it valid."""
    return any(valid_bound(bind(prog, m)) for m in memberships(prog))


# ----------------------------------------------------------------------------------------------- cost (Section 5.2)
def machine(name: str) -> dict:
    """Bandwidths in GB/s.  The H100 and V100 figures reproduce the completion times the paper prints for its three
    examples; the A100 and B200 entries follow the same model with those parts' nominal figures (not pinned by the paper)."""
    if name == "dgx_h100":
        return {"kind": "nvswitch", "n": 8, "link": 450.0, "hbm": 3350.0}
    if name == "dgx_a100":
        return {"kind": "nvswitch", "n": 8, "link": 300.0, "hbm": 2039.0}
    if name == "hgx_b200":
        return {"kind": "nvswitch", "n": 8, "link": 900.0, "hbm": 7700.0}
    if name == "dgx_v100":
        return {"kind": "cube_mesh", "n": 8, "double": 50.0, "single": 25.0, "pcie": 15.75, "hbm": 900.0}
    raise ValueError(name)


def _link(mach, a, b):
    """("link", capacity) of the direct link a -> b of the cube mesh (or of a machine given as a table of directed links,
    {"kind": "links", "links": [[GB/s]], "pcie": bridge, "hbm": ...}), or ("pcie", capacity)."""
    if mach["kind"] == "links":
        c = mach["links"][a][b]
        return ("link", c) if c > 0 else ("pcie", mach["pcie"])
    if abs(a - b) == 4:
        return ("link", mach["double"])
    if a // 4 == b // 4:
        return ("link", mach["single"])
    return ("pcie", mach["pcie"])


def simulate(prog: Program, mach: dict, trace: bool = False):
    """Completion time in milliseconds (and, with trace, per expanded action its (start, aggregated, finished) times)."""
    acts = expanded(prog)
    size = {a: gb for a, (_, gb) in prog.atoms.items()}
    have = {}                                   # site -> {aggregate: time}
    for a, (s, _) in prog.atoms.items():
        have.setdefault(s, {})[frozenset([a])] = 0.0
    WAIT, AGG, XFER, DONE = range(4)
    st = [WAIT] * len(acts)
    rem_agg = [0.0] * len(acts)
    flows = []                                   # [action, destination, remaining GB]
    times = [[None, None, None] for _ in acts]
    now = 0.0
    while True:
        progress = True
        while progress:                          # start everything that is enabled now (zero-cost steps may enable more)
            progress = False
            for i, (x, s, d) in enumerate(acts):
                if st[i] != WAIT:
                    continue
                cover = exact_cover(x, list(have.get(s, {})))
                if cover is None:
                    continue
                times[i][0] = now
                progress = True
                if len(cover) >= 2:
                    st[i] = AGG
                    rem_agg[i] = (len(cover) + 1) * size[next(iter(x))]
                else:
                    times[i][1] = now
                    if d:
                        st[i] = XFER
                        flows.extend([i, t, size[next(iter(x))]] for t in d)
                    else:
                        st[i] = DONE
                        times[i][2] = now
        active_agg = [i for i in range(len(acts)) if st[i] == AGG]
        if not active_agg and not flows:
            break
        per_site = {}
        for i in active_agg:
            per_site[acts[i][1]] = per_site.get(acts[i][1], 0) + 1
        rate_agg = {i: mach["hbm"] / per_site[acts[i][1]] for i in active_agg}
        rate_flow = []
        if mach["kind"] == "nvswitch":
            out_n, in_n = {}, {}
            for i, t, _ in flows:
                out_n[acts[i][1]] = out_n.get(acts[i][1], 0) + 1
                in_n[t] = in_n.get(t, 0) + 1
            rate_flow = [min(mach["link"] / out_n[acts[i][1]], mach["link"] / in_n[t]) for i, t, _ in flows]
        else:
            on = {}
            for i, t, _ in flows:
                kind, _cap = _link(mach, acts[i][1], t)
                key = "pcie" if kind == "pcie" else (acts[i][1], t)
                on[key] = on.get(key, 0) + 1
            for i, t, _ in flows:
                kind, cap = _link(mach, acts[i][1], t)
                rate_flow.append(cap / on["pcie" if kind == "pcie" else (acts[i][1], t)])
        dt = min([rem_agg[i] / rate_agg[i] for i in active_agg] + [f[2] / r for f, r in zip(flows, rate_flow)])
        now += dt
        for i in active_agg:
            rem_agg[i] -= rate_agg[i] * dt
        for f, r in zip(flows, rate_flow):
            f[2] -= r * dt
        eps = 1e-12
        keep = []
        for f, r in zip(flows, rate_flow):
            if f[2] <= eps * (1.0 + r * dt):
                have.setdefault(f[1], {}).setdefault(acts[f[0]][0], now)
            else:
                keep.append(f)
        flows = keep
        for i in active_agg:
            if rem_agg[i] <= eps * (1.0 + rate_agg[i] * dt):
                x, s, d = acts[i]
                have.setdefault(s, {}).setdefault(x, now)
                times[i][1] = now
                if d:
                    st[i] = XFER
                    flows.extend([i, t, size[next(iter(x))]] for t in d)
                else:
                    st[i] = DONE
                    times[i][2] = now
        for i in range(len(acts)):
            if st[i] == XFER and not any(f[0] == i for f in flows):
                st[i] = DONE
                times[i][2] = now
    if any(s != DONE for s in st):
        raise ValueError("the program is not well-formed: an action never becomes enabled")
    ms = now * 1e3                                # GB / (GB/s) = s
    return (ms, [(acts[i], tuple(None if t is None else t * 1e3 for t in times[i])) for i in range(len(acts))]) if trace else ms


# -------------------------------------------------------------------------------- bodies: the trivial valid program
def naive_body(prog: Program) -> Program:
    """Section 5.4: gather the atoms of each required aggregate at each of its target sites and aggregate there.
    One multicast per atom (all the sites that need it), one local aggregation per requirement."""
    q = prog.copy()
    q.actions = []
    need = {}                                    # atom -> destinations
    for x, s in requirements(prog):
        for a in x:
            if prog.atoms[a][0] != s:
                need.setdefault(a, set()).add(s)
    for a in prog.atoms:
        if a in need:
            q.actions.append((frozenset([a]), ("sites", (prog.atoms[a][0],)), tuple(sorted(need[a]))))
    for x, t in prog.out:
        if len(x) > 1:
            act = (x, t, ())
            if act not in q.actions:
                q.actions.append(act)
    return q


def butterfly_body(prog: Program) -> Program:
    """Recursive doubling (the pattern of Example "Recursive doubling") for every required aggregate whose targets are exactly
    the sites that hold its atoms, 2^k of them with equally many atoms each: in round b the site at position i of the
    ascending target list sends what it has aggregated so far to the site at position i xor 2^b.  Other requirements are
    served as in naive_body.  Memberships must be bound."""
    q = prog.copy()
    q.actions = []
    order = _name_order(prog)

    def add(act):
        if act not in q.actions:
            q.actions.append(act)

    groups = {}
    for x, s in requirements(prog):
        groups.setdefault(x, set()).add(s)
    need = {}
    local = []
    for x, targets in groups.items():
        t = sorted(targets)
        held = {s: frozenset(a for a in x if prog.atoms[a][0] == s) for s in t}
        k = len(t).bit_length() - 1
        ok = (len(t) >= 2 and (1 << k) == len(t) and {prog.atoms[a][0] for a in x} == set(t)
              and len({len(h) for h in held.values()}) == 1)
        if not ok:
            for s in t:
                for a in sorted(x, key=order.get):
                    if prog.atoms[a][0] != s:
                        need.setdefault(a, set()).add(s)
            if len(x) > 1:
                local.append((x, tuple(t)))
            continue
        cur = [held[s] for s in t]
        for b in range(k):
            for i, s in enumerate(t):
                add((cur[i], ("sites", (s,)), (t[i ^ (1 << b)],)))
            cur = [cur[i] | cur[i ^ (1 << b)] for i in range(len(t))]
        local.append((x, tuple(t)))
    for a in prog.atoms:
        if a in need:
            add((frozenset([a]), ("sites", (prog.atoms[a][0],)), tuple(sorted(need[a]))))
    for x, t in local:
        add((x, ("sites", t), ()))
    return q


def place(prog: Program, mach: dict, body=None, enumeration_limit: int = 5000):
    """Choose the members of the size-declared partitions: among the memberships under which the program (its own body,
    or body(bound preamble) if a synthesiser is given) is valid, the one with the least simulated completion time, among
    equal times the one that sends the fewest bytes, then the first in enumeration order.  Above `enumeration_limit` memberships: steepest descent over exchanges of two sites
    between two partitions instead.  Returns (membership, bound program, milliseconds)."""
    def cost(m):
        q = bind(prog, m)
        if body is not None:
            q = body(q)
        if not valid_bound(q):
            return None
        moved = sum(q.atoms[next(iter(x))][1] * len(d) for x, _, d in expanded(q))
        return (m, q, simulate(q, mach), moved)

    def better(c, ref):      # less simulated time; among equal times, fewer bytes sent
        if ref is None:
            return True
        if c[2] < ref[2] * (1.0 - 1e-12):
            return True
        return c[2] <= ref[2] * (1.0 + 1e-12) and c[3] < ref[3] * (1.0 - 1e-12)

    names = [n for n, p in prog.partitions.items() if p["members"] is None]
    taken = {s for p in prog.partitions.values() if p["members"] is not None for s in p["members"]}
    n_free = len([s for s in prog.gpus if s not in taken])
    total = 1
    for n in names:
        k = prog.partitions[n]["size"]
        total *= math.comb(n_free, k)
        n_free -= k
    best = None
    if total <= enumeration_limit:
        for m in memberships(prog):
            c = cost(m)
            if c is not None and better(c, best):
                best = c
    else:
        # steepest descent over exchanges of two sites between partitions, from the first membership in enumeration order
        free = [s for s in prog.gpus if s not in taken]
        cur, at = {}, 0
        for n in names:
            cur[n] = tuple(free[at: at + prog.partitions[n]["size"]])
            at += prog.partitions[n]["size"]
        best = cost(cur)
        improved = True
        while improved:
            improved = False
            pick = None
            for ia, a in enumerate(names):
                for b in names[ia + 1:]:
                    for i in range(len(cur[a])):
                        for j in range(len(cur[b])):
                            nxt = dict(cur)
                            la, lb = list(cur[a]), list(cur[b])
                            la[i], lb[j] = lb[j], la[i]
                            nxt[a], nxt[b] = tuple(la), tuple(lb)
                            c = cost(nxt)
                            if c is None:
                                continue
                            if better(c, pick if pick is not None else best):
                                pick = (nxt, c[1], c[2], c[3])
            if pick is not None:
                cur = pick[0]
                best = ({n: tuple(sorted(v)) for n, v in pick[0].items()}, pick[1], pick[2], pick[3])
                improved = True
    if best is None:
        raise ValueError("no membership makes the program valid")
    return best[:3]


# ----------------------------------------------------------------------------------- preamble generation (Section 5.3)
def preamble(extents, producer_splits, copy_site, consumer_splits, consumer_specs, width_bytes, name=None) -> Program:
    """The preamble that links a compiled producer to one input of `op`.
    producer_splits / consumer_splits: per dimension the split points of out(J_k) and of in_k(J).
    copy_site[(producer block, c)] = GPU holding copy c of that block (blocks are flat keys in row-major key order).
    consumer_specs: for every function spec of op, the flat key of the in_k block it consumes.
    Atoms = cells of the overlay of the two tilings, numbered in row-major order; IN has one ExProg atom per (atom, copy);
    PARTITIONS one partition of size one per function spec; OUT the aggregate of an atom's copies at the partition of every
    function spec whose input block contains the atom."""
    rank = len(extents)
    over = [sorted(set(producer_splits[d]) | set(consumer_splits[d])) for d in range(rank)]

    def owner(splits, lo):
        for i in range(len(splits) - 1):
            if splits[i] <= lo < splits[i + 1]:
                return i
        raise ValueError

    def flat(splits_all, lows):
        k = 0
        for d in range(rank):
            k = k * (len(splits_all[d]) - 1) + owner(splits_all[d], lows[d])
        return k

    name = name or (lambda j, c: "a%d_%d" % (j, c))
    copies = {}
    for (blk, c) in copy_site:
        copies.setdefault(blk, []).append(c)
    prog = Program(sorted(set(copy_site.values()) | set(range(len(consumer_specs)))))
    for i in range(len(consumer_specs)):
        prog.partitions["S%d" % (i + 1)] = {"size": 1, "members": None}
    cells = list(itertools.product(*[range(len(o) - 1) for o in over]))
    per_atom = []
    for j, cell in enumerate(cells):
        lows = [over[d][cell[d]] for d in range(rank)]
        card = 1
        for d in range(rank):
            card *= over[d][cell[d] + 1] - over[d][cell[d]]
        pb, cb = flat(producer_splits, lows), flat(consumer_splits, lows)
        per_atom.append((j, pb, cb, card * width_bytes / 1e9))
    # IN in site order, then atom order inside a site (the order the printed example uses)
    entries = [(copy_site[(pb, c)], j, c, gb) for j, pb, cb, gb in per_atom for c in sorted(copies[pb])]
    for site, j, c, gb in sorted(entries):
        prog.atoms[name(j, c)] = (site, gb)
    for j, pb, cb, gb in per_atom:
        x = frozenset(name(j, c) for c in copies[pb])
        for i, blk in enumerate(consumer_specs):
            if blk == cb:
                prog.out.append((x, ("part", "S%d" % (i + 1))))
    if len(prog.gpus) != len(consumer_specs):
        raise ValueError("one function spec of op per GPU: the partitions of size one must cover the GPUs")
    _check_static(prog)
    return prog


# ------------------------------------------------------------------------------------- rewriting rules (Section 5.4)
# Every rule works on a program whose memberships are bound and whose actions are written with one source site
# ("sites", (s,)); it returns the rewritten program, or None when its guard (the result must be valid) fails.
def normalised(prog: Program) -> Program:
    q = prog.copy()
    q.actions = [(x, ("sites", (s,)), d) for x, s, d in expanded(prog)]
    return q


def _guarded(q: Program):
    return q if valid_bound(q) else None


def insert(prog, action):
    """Insert(a): permitted whenever the result is well-formed."""
    q = prog.copy()
    if action not in q.actions:
        q.actions.append(action)
    return q if well_formed(q) else None


def delete(prog, index):
    """Delete(a): permitted whenever the result is valid."""
    q = prog.copy()
    del q.actions[index]
    return _guarded(q)


def fission(prog, index, part):
    """X @ s -> D1 u D2  =>  X @ s -> D1 and X @ s -> D2."""
    x, src, d = prog.actions[index]
    d1 = tuple(t for t in d if t in part)
    d2 = tuple(t for t in d if t not in part)
    if not d1 or not d2:
        return None
    q = prog.copy()
    q.actions[index] = (x, src, d1)
    q.actions.append((x, src, d2))
    return _guarded(q)


def fusion(prog, i, j):
    """X @ s -> D1 and X @ s -> D2  =>  X @ s -> D1 u D2."""
    (x, src, d1), (y, src2, d2) = prog.actions[i], prog.actions[j]
    if i == j or x != y or src != src2 or not d1 or not d2:
        return None
    q = prog.copy()
    q.actions[i] = (x, src, tuple(sorted(set(d1) | set(d2))))
    del q.actions[j]
    return _guarded(q)


def relay_introduction(prog, index, dest, relay):
    """X @ s -> d  =>  X @ s -> r and X @ r -> d."""
    x, src, d = prog.actions[index]
    if dest not in d or relay == src[1][0] or relay in d or relay not in prog.gpus:
        return None
    q = prog.copy()
    rest = tuple(t for t in d if t != dest)
    q.actions[index] = (x, src, tuple(sorted(rest + (relay,))))
    hop = (x, ("sites", (relay,)), (dest,))
    if hop not in q.actions:
        q.actions.append(hop)
    return _guarded(q)


def relay_elimination(prog, i, j):
    """X @ s -> r and X @ r -> d  =>  X @ s -> d   (only if X at r is not otherwise required: the guard)."""
    (x, src, d1), (y, src2, d2) = prog.actions[i], prog.actions[j]
    r = src2[1][0]
    if i == j or x != y or d1 != (r,) or len(d2) != 1:
        return None
    q = prog.copy()
    q.actions[i] = (x, src, d2)
    del q.actions[j]
    return _guarded(q)


def pushdown(prog, i, j):
    """X @ r -> s and Y @ r -> s  =>  X+Y @ r -> s   (eager partial aggregation)."""
    (x, src, d1), (y, src2, d2) = prog.actions[i], prog.actions[j]
    if i == j or src != src2 or d1 != d2 or not d1 or x & y:
        return None
    if len({prog.atoms[a][1] for a in x | y}) != 1:
        return None
    q = prog.copy()
    q.actions[i] = (x | y, src, d1)
    del q.actions[j]
    return _guarded(q)


def pullup(prog, index, part, restore=True):
    """X+Y @ r -> s  =>  X @ r -> s and Y @ r -> s, with the local aggregation X+Y @ s put back if `restore`."""
    xy, src, d = prog.actions[index]
    x = frozenset(part)
    y = xy - x
    if not d or not x or not y or not x < xy:
        return None
    q = prog.copy()
    q.actions[index] = (x, src, d)
    q.actions.append((y, src, d))
    if restore:
        for t in d:
            loc = (xy, ("sites", (t,)), ())
            if loc not in q.actions:
                q.actions.append(loc)
    return _guarded(q)


def source_substitution(prog, index, site):
    """Redirect the transfer of X to draw from another site at which X is materialised."""
    x, src, d = prog.actions[index]
    if not d or site == src[1][0] or site in d or (x, site) not in closure(prog):
        return None
    q = prog.copy()
    q.actions[index] = (x, ("sites", (site,)), d)
    return _guarded(q)


def neighbours(prog: Program):
    """Every program one rule application away from `prog` (bound memberships, one source site per action), guards applied."""
    p = normalised(prog)
    n = len(p.actions)
    state = closure(p)
    res = []

    def add(q):
        if q is not None:
            res.append(q)

    for i in range(n):
        x, src, d = p.actions[i]
        add(delete(p, i))
        if len(d) > 1:
            for t in d:
                add(fission(p, i, (t,)))
        if d:
            for s in p.gpus:
                if (x, s) in state:
                    add(source_substitution(p, i, s))
            for t in d:
                for r in p.gpus:
                    add(relay_introduction(p, i, t, r))
            if len(x) > 1:
                order = _name_order(p)
                for a in sorted(x, key=order.get):
                    add(pullup(p, i, (a,)))
        for j in range(n):
            if j != i:
                add(relay_elimination(p, i, j))
            if j > i:
                add(fusion(p, i, j))
                add(pushdown(p, i, j))
    return res


def _key(prog):
    order = _name_order(prog)
    return tuple(sorted((tuple(sorted(order[a] for a in x)), s, tuple(sorted(d))) for x, s, d in expanded(prog)))


def synthesize(prog: Program, mach: dict, depth: int = 6, beam: int = 24):
    """A body for a bound preamble: beam search from the better of two constructed programs (gather everything; recursive
    doubling where it applies) -- or from the program's own body if it has one -- through the rewriting rules, every candidate
    checked by Definition "Closure; validity" and costed by the simulator.  Returns (program, milliseconds).  The paper leaves
    the search procedure open; this one only has to stay inside the space of valid programs and never return a program slower
    than the trivial one."""
    if prog.actions:
        cands = [normalised(prog)]
    else:
        cands = [normalised(naive_body(prog)), normalised(butterfly_body(prog))]
    best = min(((simulate(c, mach), c) for c in cands), key=lambda t: t[0])      # the first of equals
    start = best[1]
    level = [best]
    seen = {_key(start)}
    for _ in range(depth):
        nxt = []
        for _, q in level:
            for r in neighbours(q):
                k = _key(r)
                if k in seen:
                    continue
                seen.add(k)
                nxt.append((simulate(r, mach), r))
        if not nxt:
            break
        nxt.sort(key=lambda t: (t[0], len(t[1].actions)))
        level = nxt[:beam]
        if level[0][0] < best[0] * (1.0 - 1e-12):
            best = level[0]
    return best[1], best[0]


# ------------------------------------------------------------------ executing a program over tensors (Sections 5.1 - 5.3)
def schedule(prog: Program):
    """A firing order of a valid bound program and, per fired action, the parts it aggregates: repeated passes over the
    expanded actions in body order, an action fires the first time aggregates at its source partition its aggregate
    (the partition with the fewest parts; candidates tried in ascending order of their atom masks, so the parts come out
    in ascending order of their first atoms).  Returns [(aggregate, site, destinations, [parts])]."""
    order = _name_order(prog)

    def mask(y):
        return sum(1 << order[a] for a in y)

    have = {}
    for a, (s, _) in prog.atoms.items():
        have.setdefault(s, set()).add(frozenset([a]))
    acts = expanded(prog)
    fired = [False] * len(acts)
    res = []
    progress = True
    while progress:
        progress = False
        for i, (x, s, d) in enumerate(acts):
            if fired[i]:
                continue
            cover = exact_cover(x, sorted(have.get(s, ()), key=mask), order)
            if cover is None:
                continue
            fired[i] = True
            progress = True
            res.append((x, s, d, cover))
            have.setdefault(s, set()).add(x)
            for t in d:
                have.setdefault(t, set()).add(x)
    if not all(fired):
        raise ValueError("the program is not well-formed")
    return res


def execute(prog: Program, values: dict, agg: str = "sum", dtype=None, combine=None):
    """Runs a valid bound program on tensors: values[atom name] = array.  Every fired action materialises its aggregate at
    its source -- the (+)-combination of its parts in the order `schedule` gives, in fp64, rounded once to `dtype` -- and
    copies it to its destinations.  Returns {(aggregate, site): array}.  `combine(parts) -> array` replaces the fp64
    combination (a test restates the same order in another precision with it)."""
    import numpy as np

    from . import core

    def default(parts):
        acc = np.asarray(parts[0], dtype=np.float64).copy()
        for p in parts[1:]:
            acc = acc + p if agg == "sum" else np.maximum(acc, p)
        return core.round_to(acc, dtype) if dtype in ("f32", "bf16", "f16") else acc

    if agg not in ("sum", "max"):
        raise ValueError(agg)
    combine = combine or default
    store = {(frozenset([a]), s): values[a] for a, (s, _) in prog.atoms.items()}
    for x, s, d, cover in schedule(prog):
        if len(cover) >= 2:
            store[(x, s)] = combine([store[(y, s)] for y in cover])
        for t in d:
            store.setdefault((x, t), store[(x, s)])
    return store


def exchange(prog: Program, partials, producer_splits, consumer_splits, consumer_specs, agg="sum", dtype=None,
             combine=None, name=None):
    """Section 5.3 end to end for one input of op: decompose (every resident copy of a producer block is sliced into its
    atoms), the exchange program, recompose (the aggregated atoms delivered to the GPU of function spec i are concatenated
    into the block it consumes).  `partials` is the dense tensor P[c, x...] whose copy c of producer block b is the slice
    of P[c] over that block; `prog` a valid bound program over the preamble `preamble(...)` generates for these tilings.
    Returns the dense tensor assembled from the blocks of all function specs (for a block consumed by several specs, the
    lowest one's) -- NaN where no spec consumes."""
    import numpy as np

    name = name or (lambda j, c: "a%d_%d" % (j, c))
    P = np.asarray(partials)
    m = P.shape[0]
    rank = P.ndim - 1
    over = [sorted(set(producer_splits[d]) | set(consumer_splits[d])) for d in range(rank)]
    cells = list(itertools.product(*[range(len(o) - 1) for o in over]))
    boxes = [tuple(slice(over[d][cell[d]], over[d][cell[d] + 1]) for d in range(rank)) for cell in cells]
    values = {name(j, c): P[(c,) + boxes[j]] for j in range(len(cells)) for c in range(m) if name(j, c) in prog.atoms}
    store = execute(prog, values, agg, dtype, combine)
    out = np.full(P.shape[1:], np.nan)
    done = set()

    def cblock(j):
        k = 0
        for d in range(rank):
            lo = over[d][cells[j][d]]
            idx = max(i for i in range(len(consumer_splits[d]) - 1) if consumer_splits[d][i] <= lo)
            k = k * (len(consumer_splits[d]) - 1) + idx
        return k

    for i, blk in enumerate(consumer_specs):
        site = prog.partitions["S%d" % (i + 1)]["members"][0]
        for j in range(len(cells)):
            if cblock(j) != blk or j in done:
                continue
            x = frozenset(name(j, c) for c in range(m))
            out[boxes[j]] = store[(x, site)]
            done.add(j)
    return out
