// Exchange programs (Section 5): the ExProg language of Section 5.2, Definition "Closure; validity" and the rewriting
// rules of Section 5.4, the cost model of the hardware simulator, preamble generation of Section 5.3. Host code only.
//
// An aggregate is a 64-bit mask over the atoms in declaration order, a state a set of (mask, site) pairs. A program is a
// SET of actions; wherever an order is needed it is the order of the text.
#include <ctype.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <charconv>
#include <map>
#include <mutex>
#include <set>
#include <string>
#include <tuple>
#include <utility>
#include <vector>

#include "ja_exprog.h"
#include "ja_internal.h"

struct ExTarget {
    int part = -1;                 // >= 0: a partition, else the list of sites
    std::vector<int> sites;
    bool operator==(const ExTarget& o) const { return part == o.part && sites == o.sites; }
};
struct ExAction {
    uint64_t agg = 0;
    ExTarget src;
    std::vector<int> dests;
    bool operator==(const ExAction& o) const { return agg == o.agg && src == o.src && dests == o.dests; }
};
struct ExPartition {
    std::string name;
    int size = 0;
    bool bound = false;
    std::vector<int> members;
};
struct ExAtom {
    std::string name;
    int site = 0;
    double gb = 1.0;
};
struct ja_exprog {
    std::vector<int> gpus;
    std::vector<ExPartition> parts;
    std::vector<ExAtom> atoms;
    std::vector<std::pair<uint64_t, ExTarget>> out;
    std::vector<ExAction> actions;
};

namespace {

typedef ja_exprog Prog;
struct Flat {              // an expanded action
    uint64_t agg;
    int site;
    std::vector<int> dests;
    bool operator==(const Flat& o) const { return agg == o.agg && site == o.site && dests == o.dests; }
};
typedef std::set<std::pair<int, uint64_t>> State;    // (site, aggregate)

// ------------------------------------------------------------------------------------------------------ text
std::string trim(const std::string& s) {
    size_t a = s.find_first_not_of(" \t\r\n"), b = s.find_last_not_of(" \t\r\n");
    return a == std::string::npos ? std::string() : s.substr(a, b - a + 1);
}
std::vector<std::string> split(const std::string& s, const char* seps) {
    std::vector<std::string> res;
    std::string cur;
    for (char c : s) {
        if (strchr(seps, c)) {
            res.push_back(cur);
            cur.clear();
        } else {
            cur.push_back(c);
        }
    }
    res.push_back(cur);
    return res;
}
bool is_word(const std::string& s) {
    if (s.empty()) return false;
    for (char c : s)
        if (!(isalnum((unsigned char)c) || c == '_')) return false;
    return true;
}
bool parse_int(const std::string& t, int* v) {
    std::string s = trim(t);
    if (s.empty() || s.size() > 9) return false;
    for (char c : s)
        if (!isdigit((unsigned char)c)) return false;
    *v = atoi(s.c_str());
    return true;
}
bool parse_sites(const std::string& text, std::vector<int>* sites) {
    sites->clear();
    for (const std::string& t : split(text, ",")) {
        if (trim(t).empty()) continue;
        int v;
        if (!parse_int(t, &v)) return false;
        sites->push_back(v);
    }
    return true;
}
std::vector<std::string> items(const std::string& text) {
    std::vector<std::string> res;
    for (const std::string& t : split(text, ";\n"))
        if (!trim(t).empty()) res.push_back(trim(t));
    return res;
}
int find_part(const Prog& p, const std::string& name) {
    for (size_t i = 0; i < p.parts.size(); ++i)
        if (p.parts[i].name == name) return (int)i;
    return -1;
}
int find_atom(const Prog& p, const std::string& name) {
    for (size_t i = 0; i < p.atoms.size(); ++i)
        if (p.atoms[i].name == name) return (int)i;
    return -1;
}
bool parse_target(const Prog& p, const std::string& text, ExTarget* t) {
    std::string s = trim(text);
    t->part = find_part(p, s);
    t->sites.clear();
    if (t->part >= 0) return true;
    return parse_sites(s, &t->sites) && !t->sites.empty();
}
bool parse_aggregate(const Prog& p, const std::string& text, uint64_t* mask) {
    *mask = 0;
    for (const std::string& t : split(text, "+")) {
        int a = find_atom(p, trim(t));
        if (a < 0 || (*mask >> a) & 1) return false;
        *mask |= 1ull << a;
    }
    return *mask != 0;
}
// position of keyword "KW:" (KW preceded by a non-word character, optional blanks before the colon); npos if absent
size_t find_keyword(const std::string& s, const char* kw, size_t from, size_t* after) {
    size_t n = strlen(kw);
    for (size_t i = s.find(kw, from); i != std::string::npos; i = s.find(kw, i + 1)) {
        if (i > 0 && (isalnum((unsigned char)s[i - 1]) || s[i - 1] == '_')) continue;
        size_t j = i + n;
        while (j < s.size() && (s[j] == ' ' || s[j] == '\t')) ++j;
        if (j < s.size() && s[j] == ':') {
            *after = j + 1;
            return i;
        }
    }
    return std::string::npos;
}

ja_status_t check_static(const Prog& p) {
    std::set<int> g(p.gpus.begin(), p.gpus.end());
    if (g.size() != p.gpus.size()) return ja_fail(JA_ERR_INVALID_ARG, "a site is listed twice in GPUS");
    for (int s : p.gpus)
        if (s < 0 || s > 63) return ja_fail(JA_ERR_INVALID_ARG, "site %d: sites are 0..63", s);
    std::set<int> fixed;
    int total = 0;
    for (const ExPartition& q : p.parts) {
        total += q.size;
        if (!q.bound) continue;
        for (int s : q.members) {
            if (!g.count(s) || !fixed.insert(s).second)
                return ja_fail(JA_ERR_INVALID_ARG, "partitions overlap or name an undeclared site (%s)", q.name.c_str());
        }
    }
    if (!p.parts.empty() && total != (int)p.gpus.size())
        return ja_fail(JA_ERR_INVALID_ARG, "the partitions must cover the declared GPUs");
    for (const ExAtom& a : p.atoms)
        if (!g.count(a.site)) return ja_fail(JA_ERR_INVALID_ARG, "atom %s at an undeclared site", a.name.c_str());
    auto sized = [&](uint64_t m) {
        double gb = -1.0;
        for (size_t i = 0; i < p.atoms.size(); ++i)
            if ((m >> i) & 1) {
                if (gb >= 0 && p.atoms[i].gb != gb) return false;
                gb = p.atoms[i].gb;
            }
        return true;
    };
    for (const auto& o : p.out) {
        if (!sized(o.first)) return ja_fail(JA_ERR_INVALID_ARG, "the atoms of one aggregate differ in size");
        for (int t : o.second.sites)
            if (!g.count(t)) return ja_fail(JA_ERR_INVALID_ARG, "OUT names the undeclared site %d", t);
    }
    for (const ExAction& a : p.actions) {
        if (!sized(a.agg)) return ja_fail(JA_ERR_INVALID_ARG, "the atoms of one aggregate differ in size");
        for (int t : a.src.sites)
            if (!g.count(t)) return ja_fail(JA_ERR_INVALID_ARG, "an action names the undeclared site %d", t);
        for (int t : a.dests)
            if (!g.count(t)) return ja_fail(JA_ERR_INVALID_ARG, "an action names the undeclared site %d", t);
    }
    return JA_OK;
}

ja_status_t parse_program(const std::string& text, Prog* p) {
    size_t out_after = 0, out_at = find_keyword(text, "OUT", 0, &out_after);
    if (out_at == std::string::npos) return ja_fail(JA_ERR_PARSE, "no OUT declaration");
    // the body starts after the first blank line that follows OUT
    size_t pre_end = text.size(), body_at = text.size();
    for (size_t i = text.find('\n', out_after); i != std::string::npos; i = text.find('\n', i + 1)) {
        size_t j = i + 1;
        while (j < text.size() && (text[j] == ' ' || text[j] == '\t')) ++j;
        if (j < text.size() && text[j] == '\n') {
            pre_end = i;
            body_at = j + 1;
            break;
        }
    }
    const std::string pre = text.substr(0, pre_end), body = text.substr(body_at);
    struct Mark {
        size_t at, after;
        int kw;
    };
    static const char* const KW[4] = {"GPUS", "PARTITIONS", "IN", "OUT"};
    std::vector<Mark> marks;
    for (int k = 0; k < 4; ++k) {
        size_t after = 0, from = 0, at;
        while ((at = find_keyword(pre, KW[k], from, &after)) != std::string::npos) {
            marks.push_back({at, after, k});
            from = at + 1;
        }
    }
    std::sort(marks.begin(), marks.end(), [](const Mark& a, const Mark& b) { return a.at < b.at; });
    std::string sect[4];
    bool has[4] = {false, false, false, false};
    for (size_t i = 0; i < marks.size(); ++i) {
        size_t end = i + 1 < marks.size() ? marks[i + 1].at : pre.size();
        sect[marks[i].kw] = pre.substr(marks[i].after, end - marks[i].after);
        has[marks[i].kw] = true;
    }
    if (!has[2]) return ja_fail(JA_ERR_PARSE, "no IN declaration");
    // PARTITIONS: name { size n } | name { s, s, .. }
    {
        const std::string& s = sect[1];
        size_t i = 0;
        while ((i = s.find('{', i)) != std::string::npos) {
            size_t close = s.find('}', i);
            if (close == std::string::npos) return ja_fail(JA_ERR_PARSE, "PARTITIONS: missing '}'");
            size_t b = i;
            while (b > 0 && (s[b - 1] == ' ' || s[b - 1] == '\t')) --b;
            size_t a = b;
            while (a > 0 && (isalnum((unsigned char)s[a - 1]) || s[a - 1] == '_')) --a;
            ExPartition q;
            q.name = s.substr(a, b - a);
            if (!is_word(q.name)) return ja_fail(JA_ERR_PARSE, "PARTITIONS: a partition needs a name");
            std::string inner = trim(s.substr(i + 1, close - i - 1));
            if (inner.compare(0, 4, "size") == 0 && inner.size() > 4 && (inner[4] == ' ' || inner[4] == '\t')) {
                if (!parse_int(inner.substr(4), &q.size)) return ja_fail(JA_ERR_PARSE, "PARTITIONS: bad size of %s", q.name.c_str());
            } else {
                if (!parse_sites(inner, &q.members)) return ja_fail(JA_ERR_PARSE, "PARTITIONS: bad members of %s", q.name.c_str());
                q.size = (int)q.members.size();
                q.bound = true;
            }
            p->parts.push_back(q);
            i = close + 1;
        }
    }
    for (const std::string& it : items(sect[2])) {          // IN: name @ site [(size: x GB)]
        size_t at = it.find('@');
        if (at == std::string::npos) return ja_fail(JA_ERR_PARSE, "bad IN item: %s", it.c_str());
        ExAtom a;
        a.name = trim(it.substr(0, at));
        std::string rest = trim(it.substr(at + 1));
        size_t par = rest.find('(');
        std::string site = trim(par == std::string::npos ? rest : rest.substr(0, par));
        if (!is_word(a.name) || !parse_int(site, &a.site)) return ja_fail(JA_ERR_PARSE, "bad IN item: %s", it.c_str());
        if (par != std::string::npos) {
            std::string in = trim(rest.substr(par + 1));
            if (in.empty() || in.back() != ')') return ja_fail(JA_ERR_PARSE, "bad IN item: %s", it.c_str());
            in = trim(in.substr(0, in.size() - 1));
            size_t colon = in.find(':');
            if (trim(in.substr(0, colon == std::string::npos ? 0 : colon)) != "size" || in.size() < 2 ||
                in.compare(in.size() - 2, 2, "GB") != 0)
                return ja_fail(JA_ERR_PARSE, "bad IN item: %s", it.c_str());
            std::string num = trim(in.substr(colon + 1, in.size() - 2 - colon - 1));
            char* end = nullptr;
            a.gb = strtod(num.c_str(), &end);
            if (num.empty() || *end) return ja_fail(JA_ERR_PARSE, "bad size in IN item: %s", it.c_str());
        }
        if (find_atom(*p, a.name) >= 0) return ja_fail(JA_ERR_PARSE, "atom %s declared twice", a.name.c_str());
        if (p->atoms.size() == 64) return ja_fail(JA_ERR_INVALID_ARG, "more than 64 atoms");
        p->atoms.push_back(a);
    }
    if (p->atoms.empty()) return ja_fail(JA_ERR_PARSE, "IN declares no atom");
    for (const std::string& it : items(sect[3])) {          // OUT: aggregate @ sites | partition
        size_t at = it.find('@');
        std::pair<uint64_t, ExTarget> o;
        if (at == std::string::npos || !parse_aggregate(*p, it.substr(0, at), &o.first) || !parse_target(*p, it.substr(at + 1), &o.second))
            return ja_fail(JA_ERR_PARSE, "bad OUT item: %s", it.c_str());
        p->out.push_back(o);
    }
    for (const std::string& it : items(body)) {             // aggregate @ source(s) [-> destinations]
        size_t arrow = it.find("->"), at = it.find('@');
        ExAction a;
        std::string left = arrow == std::string::npos ? it : it.substr(0, arrow);
        if (at == std::string::npos || at > left.size() || !parse_aggregate(*p, left.substr(0, at), &a.agg) ||
            !parse_target(*p, left.substr(at + 1), &a.src))
            return ja_fail(JA_ERR_PARSE, "bad action: %s", it.c_str());
        if (arrow != std::string::npos && !trim(it.substr(arrow + 2)).empty()) {
            if (!parse_sites(it.substr(arrow + 2), &a.dests)) return ja_fail(JA_ERR_PARSE, "bad action: %s", it.c_str());
            if (a.src.part >= 0 || a.src.sites.size() != 1)
                return ja_fail(JA_ERR_PARSE, "an action with an arrow has one source site: %s", it.c_str());
        }
        if (std::find(p->actions.begin(), p->actions.end(), a) == p->actions.end()) p->actions.push_back(a);   // a set
    }
    if (has[0]) {
        if (!parse_sites(sect[0], &p->gpus)) return ja_fail(JA_ERR_PARSE, "bad GPUS list");
    } else {
        std::set<int> seen;
        for (const ExAtom& a : p->atoms) seen.insert(a.site);
        for (const auto& o : p->out) seen.insert(o.second.sites.begin(), o.second.sites.end());
        for (const ExAction& a : p->actions) {
            seen.insert(a.dests.begin(), a.dests.end());
            seen.insert(a.src.sites.begin(), a.src.sites.end());
        }
        for (const ExPartition& q : p->parts) seen.insert(q.members.begin(), q.members.end());
        p->gpus.assign(seen.begin(), seen.end());
    }
    return check_static(*p);
}

std::string number(double v) {           // the shortest text that reads back to v, always with a '.' or an exponent
    char buf[64];
    auto r = std::to_chars(buf, buf + sizeof buf, v);
    std::string s(buf, r.ptr);
    if (s.find_first_of(".einf") == std::string::npos) s += ".0";
    return s;
}
std::string agg_text(const Prog& p, uint64_t m) {
    std::string s;
    for (size_t i = 0; i < p.atoms.size(); ++i)
        if ((m >> i) & 1) s += (s.empty() ? "" : "+") + p.atoms[i].name;
    return s;
}
std::string sites_text(const std::vector<int>& v) {
    std::string s;
    for (size_t i = 0; i < v.size(); ++i) s += (i ? ", " : "") + std::to_string(v[i]);
    return s;
}
std::string target_text(const Prog& p, const ExTarget& t) { return t.part >= 0 ? p.parts[t.part].name : sites_text(t.sites); }
std::string format_program(const Prog& p) {
    std::string s = "GPUS: " + sites_text(p.gpus) + "\n";
    if (!p.parts.empty()) {
        s += "PARTITIONS:";
        for (const ExPartition& q : p.parts)
            s += " " + q.name + " {" + (q.bound ? sites_text(q.members) : "size " + std::to_string(q.size)) + "}";
        s += "\n";
    }
    s += "IN: ";
    for (size_t i = 0; i < p.atoms.size(); ++i) {
        const ExAtom& a = p.atoms[i];
        s += (i ? "; " : "") + a.name + " @ " + std::to_string(a.site);
        if (a.gb != 1.0) s += " (size: " + number(a.gb) + " GB)";
    }
    s += "\nOUT: ";
    for (size_t i = 0; i < p.out.size(); ++i) s += (i ? "; " : "") + agg_text(p, p.out[i].first) + " @ " + target_text(p, p.out[i].second);
    s += "\n\n";
    for (const ExAction& a : p.actions) {
        s += agg_text(p, a.agg) + " @ " + target_text(p, a.src);
        if (!a.dests.empty()) s += " -> " + sites_text(a.dests);
        s += "\n";
    }
    return s;
}

// ------------------------------------------------------------------------------------------ memberships, expansion
bool all_bound(const Prog& p) {
    for (const ExPartition& q : p.parts)
        if (!q.bound) return false;
    return true;
}
bool resolve(const Prog& p, const ExTarget& t, std::vector<int>* sites) {
    if (t.part < 0) {
        *sites = t.sites;
        return true;
    }
    if (!p.parts[t.part].bound) return false;
    *sites = p.parts[t.part].members;
    return true;
}
bool expand(const Prog& p, std::vector<Flat>* res) {
    res->clear();
    std::vector<int> sites;
    for (const ExAction& a : p.actions) {
        if (!resolve(p, a.src, &sites)) return false;
        for (int s : sites) {
            Flat f{a.agg, s, a.dests};
            if (std::find(res->begin(), res->end(), f) == res->end()) res->push_back(f);
        }
    }
    return true;
}
bool requirements(const Prog& p, std::vector<std::pair<uint64_t, int>>* res) {
    res->clear();
    std::vector<int> sites;
    for (const auto& o : p.out) {
        if (!resolve(p, o.second, &sites)) return false;
        for (int s : sites) res->push_back({o.first, s});
    }
    return true;
}
// all memberships in enumeration order: per unbound partition (declaration order) a combination of what is left
void enumerate_memberships(const Prog& p, std::vector<std::vector<std::vector<int>>>* all) {
    std::vector<int> unbound;
    std::set<int> taken;
    for (size_t i = 0; i < p.parts.size(); ++i) {
        if (p.parts[i].bound) taken.insert(p.parts[i].members.begin(), p.parts[i].members.end());
        else unbound.push_back((int)i);
    }
    std::vector<int> free_sites;
    for (int s : p.gpus)
        if (!taken.count(s)) free_sites.push_back(s);
    std::vector<std::vector<int>> cur;
    struct Rec {
        const Prog& p;
        const std::vector<int>& unbound;
        std::vector<std::vector<std::vector<int>>>* all;
        std::vector<std::vector<int>>& cur;
        void go(size_t i, const std::vector<int>& rest) {
            if (i == unbound.size()) {
                all->push_back(cur);
                return;
            }
            const int k = p.parts[unbound[i]].size, n = (int)rest.size();
            if (k > n) return;
            std::vector<int> idx(k);
            for (int t = 0; t < k; ++t) idx[t] = t;
            while (true) {
                std::vector<int> mem, left;
                size_t q = 0;
                for (int t = 0; t < n; ++t) {
                    if (q < idx.size() && idx[q] == t) {
                        mem.push_back(rest[t]);
                        ++q;
                    } else {
                        left.push_back(rest[t]);
                    }
                }
                cur.push_back(mem);
                go(i + 1, left);
                cur.pop_back();
                int t = k - 1;
                while (t >= 0 && idx[t] == n - k + t) --t;
                if (t < 0) break;
                ++idx[t];
                for (int u = t + 1; u < k; ++u) idx[u] = idx[u - 1] + 1;
            }
        }
    } rec{p, unbound, all, cur};
    rec.go(0, free_sites);
}
void bind_membership(Prog* p, const std::vector<std::vector<int>>& mem) {
    size_t k = 0;
    for (ExPartition& q : p->parts)
        if (!q.bound) {
            q.members = mem[k++];
            std::sort(q.members.begin(), q.members.end());
            q.bound = true;
        }
}

// ---------------------------------------------------------------------------- Definition "Closure; validity"
// a partition of x into members of `avail` with the fewest parts; returns the number of parts, 0 if there is none
struct Cover {
    std::vector<uint64_t> cands;
    int best = 0;
    void rec(uint64_t rest, int parts) {
        if (best && parts >= best) return;
        if (!rest) {
            best = parts;
            return;
        }
        const uint64_t pivot = rest & (~rest + 1);
        for (uint64_t y : cands)
            if ((y & pivot) && (y & ~rest) == 0) rec(rest & ~y, parts + 1);
    }
};
// the same search, keeping the parts: candidates in the order given (callers pass them ascending), so the parts come out in
// ascending order of their first atoms and the first minimal partition found wins
struct CoverParts {
    std::vector<uint64_t> cands, cur, best;
    void rec(uint64_t rest) {
        if (!best.empty() && cur.size() >= best.size()) return;
        if (!rest) {
            best = cur;
            return;
        }
        const uint64_t pivot = rest & (~rest + 1);
        for (uint64_t y : cands)
            if ((y & pivot) && (y & ~rest) == 0) {
                cur.push_back(y);
                rec(rest & ~y);
                cur.pop_back();
            }
    }
};
int exact_cover(uint64_t x, const std::vector<uint64_t>& avail) {
    Cover c;
    for (uint64_t y : avail)
        if (y && (y & ~x) == 0) c.cands.push_back(y);
    c.rec(x, 0);
    return c.best;
}
std::vector<uint64_t> at_site(const State& st, int site) {
    std::vector<uint64_t> res;
    for (auto it = st.lower_bound({site, 0}); it != st.end() && it->first == site; ++it) res.push_back(it->second);
    return res;
}
State closure_of(const Prog& p, const std::vector<Flat>& acts) {
    State st;
    for (size_t i = 0; i < p.atoms.size(); ++i) st.insert({p.atoms[i].site, 1ull << i});
    bool changed = true;
    while (changed) {
        changed = false;
        for (const Flat& a : acts) {
            if (!exact_cover(a.agg, at_site(st, a.site))) continue;
            if (st.insert({a.site, a.agg}).second) changed = true;
            for (int d : a.dests)
                if (st.insert({d, a.agg}).second) changed = true;
        }
    }
    return st;
}
void check_bound(const Prog& p, bool* wf, bool* valid) {
    std::vector<Flat> acts;
    expand(p, &acts);
    const State st = closure_of(p, acts);
    *wf = true;
    for (const Flat& a : acts)
        if (!exact_cover(a.agg, at_site(st, a.site))) *wf = false;
    *valid = *wf;
    std::vector<std::pair<uint64_t, int>> req;
    requirements(p, &req);
    for (const auto& r : req)
        if (!st.count({r.second, r.first})) *valid = false;
}
bool valid_bound(const Prog& p) {
    bool wf, v;
    check_bound(p, &wf, &v);
    return v;
}

// --------------------------------------------------------------------------------------------------- simulator
double atom_gb(const Prog& p, uint64_t agg) {
    for (size_t i = 0; i < p.atoms.size(); ++i)
        if ((agg >> i) & 1) return p.atoms[i].gb;
    return 0.0;
}
// kind 0: a direct link of the given capacity, 1: the bridge
void mesh_link(const ja_machine_t& m, int a, int b, int* kind, double* cap) {
    if (m.fabric == JA_FABRIC_LINKS) {
        const double c = m.links[a * m.n_sites + b];
        *kind = c > 0 ? 0 : 1;
        *cap = c > 0 ? c : m.pcie_gbs;
        return;
    }
    if (abs(a - b) == 4) {
        *kind = 0;
        *cap = m.double_gbs;
    } else if (a / 4 == b / 4) {
        *kind = 0;
        *cap = m.link_gbs;
    } else {
        *kind = 1;
        *cap = m.pcie_gbs;
    }
}
struct FlowRec {
    int act, dst;
    double rem;
};
bool simulate(const Prog& p, const ja_machine_t& m, double* completion_ms, double* t_start, double* t_agg, double* t_fin) {
    std::vector<Flat> acts;
    expand(p, &acts);
    const int n = (int)acts.size();
    std::map<int, std::map<uint64_t, double>> have;
    for (size_t i = 0; i < p.atoms.size(); ++i) have[p.atoms[i].site][1ull << i] = 0.0;
    enum { WAIT, AGG, XFER, DONE };
    std::vector<int> st(n, WAIT);
    std::vector<double> rem_agg(n, 0.0), ts(n, -1.0), ta(n, -1.0), tf(n, -1.0);
    std::vector<FlowRec> flows;
    double now = 0.0;
    auto begin_transfer = [&](int i) {
        if (!acts[i].dests.empty()) {
            st[i] = XFER;
            for (int d : acts[i].dests) flows.push_back({i, d, atom_gb(p, acts[i].agg)});
        } else {
            st[i] = DONE;
            tf[i] = now;
        }
    };
    while (true) {
        bool progress = true;
        while (progress) {              // start whatever is enabled now; steps of no cost may enable more
            progress = false;
            for (int i = 0; i < n; ++i) {
                if (st[i] != WAIT) continue;
                std::vector<uint64_t> avail;
                for (const auto& kv : have[acts[i].site]) avail.push_back(kv.first);
                const int parts = exact_cover(acts[i].agg, avail);
                if (!parts) continue;
                ts[i] = now;
                progress = true;
                if (parts >= 2) {
                    st[i] = AGG;
                    rem_agg[i] = (parts + 1) * atom_gb(p, acts[i].agg);
                } else {
                    ta[i] = now;
                    begin_transfer(i);
                }
            }
        }
        std::vector<int> active;
        for (int i = 0; i < n; ++i)
            if (st[i] == AGG) active.push_back(i);
        if (active.empty() && flows.empty()) break;
        std::map<int, int> per_site;
        for (int i : active) ++per_site[acts[i].site];
        std::vector<double> rate_agg(active.size()), rate_flow(flows.size());
        for (size_t k = 0; k < active.size(); ++k) rate_agg[k] = m.hbm_gbs / per_site[acts[active[k]].site];
        if (m.fabric == JA_FABRIC_NVSWITCH) {
            std::map<int, int> out_n, in_n;
            for (const FlowRec& f : flows) {
                ++out_n[acts[f.act].site];
                ++in_n[f.dst];
            }
            for (size_t k = 0; k < flows.size(); ++k)
                rate_flow[k] = std::min(m.link_gbs / out_n[acts[flows[k].act].site], m.link_gbs / in_n[flows[k].dst]);
        } else {
            std::map<std::pair<int, int>, int> on;      // (-1, -1) = the bridge
            for (const FlowRec& f : flows) {
                int kind;
                double cap;
                mesh_link(m, acts[f.act].site, f.dst, &kind, &cap);
                ++on[kind ? std::make_pair(-1, -1) : std::make_pair(acts[f.act].site, f.dst)];
            }
            for (size_t k = 0; k < flows.size(); ++k) {
                int kind;
                double cap;
                mesh_link(m, acts[flows[k].act].site, flows[k].dst, &kind, &cap);
                rate_flow[k] = cap / on[kind ? std::make_pair(-1, -1) : std::make_pair(acts[flows[k].act].site, flows[k].dst)];
            }
        }
        double dt = INFINITY;
        for (size_t k = 0; k < active.size(); ++k) dt = std::min(dt, rem_agg[active[k]] / rate_agg[k]);
        for (size_t k = 0; k < flows.size(); ++k) dt = std::min(dt, flows[k].rem / rate_flow[k]);
        now += dt;
        for (size_t k = 0; k < active.size(); ++k) rem_agg[active[k]] -= rate_agg[k] * dt;
        for (size_t k = 0; k < flows.size(); ++k) flows[k].rem -= rate_flow[k] * dt;
        const double eps = 1e-12;
        std::vector<FlowRec> keep;
        for (size_t k = 0; k < flows.size(); ++k) {
            if (flows[k].rem <= eps * (1.0 + rate_flow[k] * dt)) {
                have[flows[k].dst].insert({acts[flows[k].act].agg, now});
            } else {
                keep.push_back(flows[k]);
            }
        }
        flows.swap(keep);
        for (size_t k = 0; k < active.size(); ++k) {
            const int i = active[k];
            if (rem_agg[i] <= eps * (1.0 + rate_agg[k] * dt)) {
                have[acts[i].site].insert({acts[i].agg, now});
                ta[i] = now;
                begin_transfer(i);
            }
        }
        for (int i = 0; i < n; ++i) {
            if (st[i] != XFER) continue;
            bool any = false;
            for (const FlowRec& f : flows) any |= f.act == i;
            if (!any) {
                st[i] = DONE;
                tf[i] = now;
            }
        }
    }
    for (int i = 0; i < n; ++i)
        if (st[i] != DONE) return false;
    *completion_ms = now * 1e3;
    for (int i = 0; i < n; ++i) {
        if (t_start) t_start[i] = ts[i] * 1e3;
        if (t_agg) t_agg[i] = ta[i] * 1e3;
        if (t_fin) t_fin[i] = tf[i] * 1e3;
    }
    return true;
}

// ------------------------------------------------------------------------------------------------------ bodies
ExTarget one_site(int s) {
    ExTarget t;
    t.sites.push_back(s);
    return t;
}
void add_action(Prog* p, const ExAction& a) {
    if (std::find(p->actions.begin(), p->actions.end(), a) == p->actions.end()) p->actions.push_back(a);
}
void naive_body(Prog* p) {
    p->actions.clear();
    std::vector<std::pair<uint64_t, int>> req;
    requirements(*p, &req);
    std::vector<std::set<int>> need(p->atoms.size());
    for (const auto& r : req)
        for (size_t a = 0; a < p->atoms.size(); ++a)
            if (((r.first >> a) & 1) && p->atoms[a].site != r.second) need[a].insert(r.second);
    for (size_t a = 0; a < p->atoms.size(); ++a) {
        if (need[a].empty()) continue;
        ExAction act;
        act.agg = 1ull << a;
        act.src = one_site(p->atoms[a].site);
        act.dests.assign(need[a].begin(), need[a].end());
        p->actions.push_back(act);
    }
    for (const auto& o : p->out) {
        if (!(o.first & (o.first - 1))) continue;      // a single atom needs no aggregation
        ExAction act;
        act.agg = o.first;
        act.src = o.second;
        add_action(p, act);
    }
}
void butterfly_body(Prog* p) {
    p->actions.clear();
    std::vector<std::pair<uint64_t, int>> req;
    requirements(*p, &req);
    std::vector<uint64_t> order;                       // aggregates in order of first appearance
    std::map<uint64_t, std::set<int>> groups;
    for (const auto& r : req) {
        if (!groups.count(r.first)) order.push_back(r.first);
        groups[r.first].insert(r.second);
    }
    std::vector<std::set<int>> need(p->atoms.size());
    std::vector<std::pair<uint64_t, std::vector<int>>> local;
    for (uint64_t x : order) {
        std::vector<int> t(groups[x].begin(), groups[x].end());
        std::vector<uint64_t> held(t.size(), 0);
        std::set<int> atom_sites;
        for (size_t a = 0; a < p->atoms.size(); ++a) {
            if (!((x >> a) & 1)) continue;
            atom_sites.insert(p->atoms[a].site);
            for (size_t i = 0; i < t.size(); ++i)
                if (t[i] == p->atoms[a].site) held[i] |= 1ull << a;
        }
        int k = 0;
        while ((2u << k) <= t.size()) ++k;
        bool ok = t.size() >= 2 && (1u << k) == t.size() && atom_sites == groups[x];
        for (size_t i = 1; ok && i < t.size(); ++i) ok = __builtin_popcountll(held[i]) == __builtin_popcountll(held[0]);
        if (!ok) {
            for (int s : t)
                for (size_t a = 0; a < p->atoms.size(); ++a)
                    if (((x >> a) & 1) && p->atoms[a].site != s) need[a].insert(s);
            if (x & (x - 1)) local.push_back({x, t});
            continue;
        }
        std::vector<uint64_t> cur = held;
        for (int b = 0; b < k; ++b) {
            for (size_t i = 0; i < t.size(); ++i) {
                ExAction act;
                act.agg = cur[i];
                act.src = one_site(t[i]);
                act.dests.push_back(t[i ^ (1u << b)]);
                add_action(p, act);
            }
            std::vector<uint64_t> nxt(t.size());
            for (size_t i = 0; i < t.size(); ++i) nxt[i] = cur[i] | cur[i ^ (1u << b)];
            cur.swap(nxt);
        }
        local.push_back({x, t});
    }
    for (size_t a = 0; a < p->atoms.size(); ++a) {
        if (need[a].empty()) continue;
        ExAction act;
        act.agg = 1ull << a;
        act.src = one_site(p->atoms[a].site);
        act.dests.assign(need[a].begin(), need[a].end());
        add_action(p, act);
    }
    for (const auto& l : local) {
        ExAction act;
        act.agg = l.first;
        act.src.sites = l.second;
        add_action(p, act);
    }
}
void normalise(Prog* p) {
    std::vector<Flat> acts;
    expand(*p, &acts);
    p->actions.clear();
    for (const Flat& f : acts) {
        ExAction a;
        a.agg = f.agg;
        a.src = one_site(f.site);
        a.dests = f.dests;
        p->actions.push_back(a);
    }
}
bool is_normal(const Prog& p) {
    for (const ExAction& a : p.actions)
        if (a.src.part >= 0 || a.src.sites.size() != 1) return false;
    return true;
}
bool same_size(const Prog& p, uint64_t m) {
    double gb = -1;
    for (size_t i = 0; i < p.atoms.size(); ++i)
        if ((m >> i) & 1) {
            if (gb >= 0 && p.atoms[i].gb != gb) return false;
            gb = p.atoms[i].gb;
        }
    return true;
}
std::vector<int> mask_sites(uint64_t m) {
    std::vector<int> v;
    for (int s = 0; s < 64; ++s)
        if ((m >> s) & 1) v.push_back(s);
    return v;
}
bool contains(const std::vector<int>& v, int s) { return std::find(v.begin(), v.end(), s) != v.end(); }

// one rule application on a normalised, bound program; q receives the rewritten program; false if the rule does not
// match or its guard fails
bool rewrite(const Prog& p, int rule, int i, int j, uint64_t a, uint64_t b, Prog* q) {
    const int n = (int)p.actions.size();
    *q = p;
    auto idx = [&](int k) { return k >= 0 && k < n; };
    switch (rule) {
    case JA_RULE_INSERT: {
        if (!a || (p.atoms.size() < 64 && (a >> p.atoms.size())) || !same_size(p, a) || !contains(p.gpus, i)) return false;
        ExAction act;
        act.agg = a;
        act.src = one_site(i);
        act.dests = mask_sites(b);
        for (int d : act.dests)
            if (!contains(p.gpus, d)) return false;
        add_action(q, act);
        bool wf, v;
        check_bound(*q, &wf, &v);
        return wf;
    }
    case JA_RULE_DELETE:
        if (!idx(i)) return false;
        q->actions.erase(q->actions.begin() + i);
        return valid_bound(*q);
    case JA_RULE_FISSION: {
        if (!idx(i)) return false;
        std::vector<int> d1, d2;
        for (int t : p.actions[i].dests) ((a >> t) & 1 ? d1 : d2).push_back(t);
        if (d1.empty() || d2.empty()) return false;
        q->actions[i].dests = d1;
        ExAction act = p.actions[i];
        act.dests = d2;
        q->actions.push_back(act);
        return valid_bound(*q);
    }
    case JA_RULE_FUSION: {
        if (!idx(i) || !idx(j) || i == j) return false;
        const ExAction &x = p.actions[i], &y = p.actions[j];
        if (x.agg != y.agg || !(x.src == y.src) || x.dests.empty() || y.dests.empty()) return false;
        std::set<int> u(x.dests.begin(), x.dests.end());
        u.insert(y.dests.begin(), y.dests.end());
        q->actions[i].dests.assign(u.begin(), u.end());
        q->actions.erase(q->actions.begin() + j);
        return valid_bound(*q);
    }
    case JA_RULE_RELAY_IN: {
        if (!idx(i)) return false;
        const ExAction& x = p.actions[i];
        const int dest = j, relay = (int)a;
        if (!contains(x.dests, dest) || relay == x.src.sites[0] || contains(x.dests, relay) || !contains(p.gpus, relay)) return false;
        std::vector<int> rest;
        for (int t : x.dests)
            if (t != dest) rest.push_back(t);
        rest.push_back(relay);
        std::sort(rest.begin(), rest.end());
        q->actions[i].dests = rest;
        ExAction hop;
        hop.agg = x.agg;
        hop.src = one_site(relay);
        hop.dests.push_back(dest);
        add_action(q, hop);
        return valid_bound(*q);
    }
    case JA_RULE_RELAY_OUT: {
        if (!idx(i) || !idx(j) || i == j) return false;
        const ExAction &x = p.actions[i], &y = p.actions[j];
        const int r = y.src.sites[0];
        if (x.agg != y.agg || x.dests.size() != 1 || x.dests[0] != r || y.dests.size() != 1) return false;
        q->actions[i].dests = y.dests;
        q->actions.erase(q->actions.begin() + j);
        return valid_bound(*q);
    }
    case JA_RULE_PUSHDOWN: {
        if (!idx(i) || !idx(j) || i == j) return false;
        const ExAction &x = p.actions[i], &y = p.actions[j];
        if (!(x.src == y.src) || x.dests != y.dests || x.dests.empty() || (x.agg & y.agg) || !same_size(p, x.agg | y.agg)) return false;
        q->actions[i].agg = x.agg | y.agg;
        q->actions.erase(q->actions.begin() + j);
        return valid_bound(*q);
    }
    case JA_RULE_PULLUP: {
        if (!idx(i)) return false;
        const ExAction& xy = p.actions[i];
        const uint64_t x = a, y = xy.agg & ~a;
        if (xy.dests.empty() || !x || !y || (x & ~xy.agg)) return false;
        q->actions[i].agg = x;
        ExAction other = xy;
        other.agg = y;
        q->actions.push_back(other);
        if (b)
            for (int t : xy.dests) {
                ExAction loc;
                loc.agg = xy.agg;
                loc.src = one_site(t);
                add_action(q, loc);
            }
        return valid_bound(*q);
    }
    case JA_RULE_SOURCE: {
        if (!idx(i)) return false;
        const ExAction& x = p.actions[i];
        if (x.dests.empty() || j == x.src.sites[0] || contains(x.dests, j)) return false;
        std::vector<Flat> acts;
        expand(p, &acts);
        if (!closure_of(p, acts).count({j, x.agg})) return false;
        q->actions[i].src = one_site(j);
        return valid_bound(*q);
    }
    }
    return false;
}

// every program one rule application away, in a fixed order (per action: delete, fissions, substitutions, relays,
// pullups; then per pair: relay elimination, fusion, pushdown)
void neighbours(const Prog& p, std::vector<Prog>* res) {
    res->clear();
    const int n = (int)p.actions.size();
    std::vector<Flat> acts;
    expand(p, &acts);
    const State st = closure_of(p, acts);
    Prog q;
    auto tryr = [&](int rule, int i, int j, uint64_t a, uint64_t b) {
        if (rewrite(p, rule, i, j, a, b, &q)) res->push_back(q);
    };
    for (int i = 0; i < n; ++i) {
        const ExAction& x = p.actions[i];
        tryr(JA_RULE_DELETE, i, 0, 0, 0);
        if (x.dests.size() > 1)
            for (int t : x.dests) tryr(JA_RULE_FISSION, i, 0, 1ull << t, 0);
        if (!x.dests.empty()) {
            for (int s : p.gpus)
                if (st.count({s, x.agg})) tryr(JA_RULE_SOURCE, i, s, 0, 0);
            for (int t : x.dests)
                for (int r : p.gpus) tryr(JA_RULE_RELAY_IN, i, t, (uint64_t)r, 0);
            if (x.agg & (x.agg - 1))
                for (size_t a = 0; a < p.atoms.size(); ++a)
                    if ((x.agg >> a) & 1) tryr(JA_RULE_PULLUP, i, 0, 1ull << a, 1);
        }
        for (int j = 0; j < n; ++j) {
            if (j != i) tryr(JA_RULE_RELAY_OUT, i, j, 0, 0);
            if (j > i) {
                tryr(JA_RULE_FUSION, i, j, 0, 0);
                tryr(JA_RULE_PUSHDOWN, i, j, 0, 0);
            }
        }
    }
}
typedef std::vector<std::tuple<uint64_t, int, std::vector<int>>> Key;
Key key_of(const Prog& p) {
    std::vector<Flat> acts;
    expand(p, &acts);
    Key k;
    for (const Flat& f : acts) {
        std::vector<int> d = f.dests;
        std::sort(d.begin(), d.end());
        k.push_back(std::make_tuple(f.agg, f.site, d));
    }
    std::sort(k.begin(), k.end());
    return k;
}
double bytes_sent(const Prog& p) {      // GB put on links: every transfer of every action
    std::vector<Flat> acts;
    expand(p, &acts);
    double gb = 0.0;
    for (const Flat& a : acts) gb += atom_gb(p, a.agg) * (double)a.dests.size();
    return gb;
}
// less simulated time; among equal times, fewer bytes sent
bool better_placement(double t, double gb, bool have_ref, double ref_t, double ref_gb) {
    if (!have_ref) return true;
    if (t < ref_t * (1.0 - 1e-12)) return true;
    return t <= ref_t * (1.0 + 1e-12) && gb < ref_gb * (1.0 - 1e-12);
}
bool best_constructed(const Prog& bound, const ja_machine_t& m, int body, Prog* best, double* ms) {
    std::vector<Prog> cands;
    if (body == JA_BODY_OWN) {
        cands.push_back(bound);
    } else {
        if (body == JA_BODY_NAIVE || body == JA_BODY_BEST) {
            cands.push_back(bound);
            naive_body(&cands.back());
        }
        if (body == JA_BODY_BUTTERFLY || body == JA_BODY_BEST) {
            cands.push_back(bound);
            butterfly_body(&cands.back());
        }
    }
    bool found = false;
    for (Prog& c : cands) {
        double t;
        if (!valid_bound(c) || !simulate(c, m, &t, nullptr, nullptr, nullptr)) continue;
        if (!found || t < *ms) {
            *best = c;
            *ms = t;
            found = true;
        }
    }
    return found;
}

ja_status_t need_bound(const Prog* p) {
    if (!p) return ja_fail(JA_ERR_INVALID_ARG, "null program");
    if (!all_bound(*p)) return ja_fail(JA_ERR_INVALID_ARG, "a partition declared by size has no members yet: bind or place the program first");
    return JA_OK;
}
ja_status_t check_machine(const ja_machine_t* m, const Prog& p) {
    if (!m) return ja_fail(JA_ERR_INVALID_ARG, "null machine");
    if (!(m->hbm_gbs > 0) || !(m->link_gbs > 0)) return ja_fail(JA_ERR_INVALID_ARG, "machine: bandwidths must be positive");
    if (m->fabric == JA_FABRIC_CUBE_MESH) {
        if (!(m->double_gbs > 0) || !(m->pcie_gbs > 0)) return ja_fail(JA_ERR_INVALID_ARG, "machine: bandwidths must be positive");
        for (int s : p.gpus)
            if (s > 7) return ja_fail(JA_ERR_INVALID_ARG, "the cube mesh has sites 0..7");
    } else if (m->fabric == JA_FABRIC_LINKS) {
        if (!m->links || m->n_sites < 1 || m->n_sites > 64) return ja_fail(JA_ERR_INVALID_ARG, "machine: a link table of n_sites x n_sites entries is needed");
        bool bridge_needed = false;
        for (int a = 0; a < m->n_sites; ++a)
            for (int b = 0; b < m->n_sites; ++b) {
                if (m->links[a * m->n_sites + b] < 0) return ja_fail(JA_ERR_INVALID_ARG, "machine: negative link capacity");
                if (a != b && m->links[a * m->n_sites + b] == 0) bridge_needed = true;
            }
        if (bridge_needed && !(m->pcie_gbs > 0)) return ja_fail(JA_ERR_INVALID_ARG, "machine: unlinked pairs need a bridge capacity");
        for (int s : p.gpus)
            if (s >= m->n_sites) return ja_fail(JA_ERR_INVALID_ARG, "site %d is not in the machine's link table", s);
    } else if (m->fabric != JA_FABRIC_NVSWITCH) {
        return ja_fail(JA_ERR_INVALID_ARG, "machine: unknown fabric");
    }
    return JA_OK;
}

}  // namespace

// memberships above this count are searched by pairwise swaps instead of being enumerated
constexpr int64_t PLACE_ENUMERATION_LIMIT = 5000;
// and above this one they are not listed at all (ja_exprog_bind by index, ja_exprog_valid_any)
constexpr int64_t MEMBERSHIP_LIST_LIMIT = 1000000;
namespace {
int64_t count_memberships(const Prog& p) {      // the multinomial, capped well above the limit
    std::set<int> taken;
    int64_t n_free = 0;
    for (const ExPartition& q : p.parts)
        if (q.bound) taken.insert(q.members.begin(), q.members.end());
    for (int s : p.gpus) n_free += !taken.count(s);
    double total = 1.0;
    for (const ExPartition& q : p.parts) {
        if (q.bound) continue;
        double c = 1.0;
        for (int i = 0; i < q.size; ++i) c = c * (double)(n_free - i) / (double)(i + 1);
        total *= c;
        n_free -= q.size;
        if (total > 1e15) return (int64_t)1e15;
    }
    return (int64_t)(total + 0.5);
}
}  // namespace

// ============================================================================================================ C ABI
extern "C" ja_status_t ja_machine_preset(const char* name, ja_machine_t* out) {
    if (!name || !out) return ja_fail(JA_ERR_INVALID_ARG, "null argument");
    ja_machine_t m = {JA_FABRIC_NVSWITCH, 8, 0, 0, 0, 0, nullptr};
    if (!strcmp(name, "dgx_h100")) {
        m.link_gbs = 450.0;
        m.hbm_gbs = 3350.0;
    } else if (!strcmp(name, "dgx_a100")) {
        m.link_gbs = 300.0;
        m.hbm_gbs = 2039.0;
    } else if (!strcmp(name, "hgx_b200")) {
        m.link_gbs = 900.0;
        m.hbm_gbs = 7700.0;
    } else if (!strcmp(name, "dgx_v100")) {
        m.fabric = JA_FABRIC_CUBE_MESH;
        m.link_gbs = 25.0;
        m.double_gbs = 50.0;
        m.pcie_gbs = 15.75;
        m.hbm_gbs = 900.0;
    } else {
        return ja_fail(JA_ERR_INVALID_ARG, "unknown machine '%s'", name);
    }
    *out = m;
    return JA_OK;
}

extern "C" ja_status_t ja_exprog_parse(const char* text, ja_exprog_t** out) {
    if (!text || !out) return ja_fail(JA_ERR_INVALID_ARG, "null argument");
    Prog* p = new Prog();
    ja_status_t st = parse_program(text, p);
    if (st != JA_OK) {
        delete p;
        return st;
    }
    *out = p;
    return JA_OK;
}
extern "C" ja_status_t ja_exprog_merge(const ja_exprog_t* a, const ja_exprog_t* b, const char* prefix_a, const char* prefix_b,
                                       ja_exprog_t** out) {
    if (!a || !b || !prefix_a || !prefix_b || !out) return ja_fail(JA_ERR_INVALID_ARG, "null argument");
    if (a->gpus != b->gpus) return ja_fail(JA_ERR_INVALID_ARG, "the two programs declare different GPUS");
    if (a->parts.size() != b->parts.size()) return ja_fail(JA_ERR_INVALID_ARG, "the two programs declare different PARTITIONS");
    for (size_t i = 0; i < a->parts.size(); ++i)
        if (a->parts[i].name != b->parts[i].name || a->parts[i].size != b->parts[i].size || a->parts[i].bound != b->parts[i].bound ||
            a->parts[i].members != b->parts[i].members)
            return ja_fail(JA_ERR_INVALID_ARG, "partition %s differs between the two programs", a->parts[i].name.c_str());
    if (a->atoms.size() + b->atoms.size() > 64) return ja_fail(JA_ERR_INVALID_ARG, "%d atoms: at most 64", (int)(a->atoms.size() + b->atoms.size()));
    Prog* p = new Prog(*a);
    const int shift = (int)a->atoms.size();
    for (ExAtom& at : p->atoms) at.name = std::string(prefix_a) + at.name;
    for (ExAtom at : b->atoms) {
        at.name = std::string(prefix_b) + at.name;
        if (!is_word(at.name) || find_atom(*p, at.name) >= 0) {
            delete p;
            return ja_fail(JA_ERR_INVALID_ARG, "atom name %s clashes or is not a word", at.name.c_str());
        }
        p->atoms.push_back(at);
    }
    for (const ExAtom& at : p->atoms)
        if (!is_word(at.name)) {
            delete p;
            return ja_fail(JA_ERR_INVALID_ARG, "atom name %s is not a word", at.name.c_str());
        }
    for (auto o : b->out) {
        o.first <<= shift;
        p->out.push_back(o);
    }
    for (ExAction act : b->actions) {
        act.agg <<= shift;
        add_action(p, act);
    }
    ja_status_t st = check_static(*p);
    if (st != JA_OK) {
        delete p;
        return st;
    }
    *out = p;
    return JA_OK;
}
extern "C" ja_status_t ja_exprog_clone(const ja_exprog_t* p, ja_exprog_t** out) {
    if (!p || !out) return ja_fail(JA_ERR_INVALID_ARG, "null argument");
    *out = new Prog(*p);
    return JA_OK;
}
extern "C" void ja_exprog_destroy(ja_exprog_t* p) { delete p; }

extern "C" ja_status_t ja_exprog_format(const ja_exprog_t* p, char* buf, int64_t cap, int64_t* needed) {
    if (!p) return ja_fail(JA_ERR_INVALID_ARG, "null program");
    const std::string s = format_program(*p);
    if (needed) *needed = (int64_t)s.size() + 1;
    if (!buf) return JA_OK;
    if (cap < (int64_t)s.size() + 1) return ja_fail(JA_ERR_INVALID_ARG, "buffer too small: %lld bytes needed", (long long)s.size() + 1);
    memcpy(buf, s.c_str(), s.size() + 1);
    return JA_OK;
}
extern "C" ja_status_t ja_exprog_counts(const ja_exprog_t* p, int32_t* n_gpus, int32_t* n_partitions, int32_t* n_atoms,
                                        int32_t* n_out, int32_t* n_actions, int32_t* n_expanded) {
    if (!p) return ja_fail(JA_ERR_INVALID_ARG, "null program");
    if (n_gpus) *n_gpus = (int32_t)p->gpus.size();
    if (n_partitions) *n_partitions = (int32_t)p->parts.size();
    if (n_atoms) *n_atoms = (int32_t)p->atoms.size();
    if (n_out) *n_out = (int32_t)p->out.size();
    if (n_actions) *n_actions = (int32_t)p->actions.size();
    if (n_expanded) {
        std::vector<Flat> acts;
        *n_expanded = expand(*p, &acts) ? (int32_t)acts.size() : -1;
    }
    return JA_OK;
}
extern "C" ja_status_t ja_exprog_get_actions(const ja_exprog_t* p, uint64_t* aggregate, int32_t* source, uint64_t* dests) {
    if (!p) return ja_fail(JA_ERR_INVALID_ARG, "null program");
    std::vector<Flat> acts;
    if (!expand(*p, &acts)) return ja_fail(JA_ERR_INVALID_ARG, "a partition used by the body has no members yet");
    for (size_t i = 0; i < acts.size(); ++i) {
        if (aggregate) aggregate[i] = acts[i].agg;
        if (source) source[i] = acts[i].site;
        if (dests) {
            dests[i] = 0;
            for (int d : acts[i].dests) dests[i] |= 1ull << d;
        }
    }
    return JA_OK;
}
extern "C" ja_status_t ja_exprog_get_requirements(const ja_exprog_t* p, int32_t* n, uint64_t* aggregate, int32_t* site) {
    if (!p) return ja_fail(JA_ERR_INVALID_ARG, "null program");
    std::vector<std::pair<uint64_t, int>> req;
    if (!requirements(*p, &req)) return ja_fail(JA_ERR_INVALID_ARG, "a partition named in OUT has no members yet");
    if (n) *n = (int32_t)req.size();
    for (size_t i = 0; i < req.size(); ++i) {
        if (aggregate) aggregate[i] = req[i].first;
        if (site) site[i] = req[i].second;
    }
    return JA_OK;
}
extern "C" ja_status_t ja_exprog_get_atoms(const ja_exprog_t* p, int32_t* site, double* size_gb) {
    if (!p) return ja_fail(JA_ERR_INVALID_ARG, "null program");
    for (size_t i = 0; i < p->atoms.size(); ++i) {
        if (site) site[i] = p->atoms[i].site;
        if (size_gb) size_gb[i] = p->atoms[i].gb;
    }
    return JA_OK;
}

extern "C" ja_status_t ja_exprog_num_memberships(const ja_exprog_t* p, int64_t* n) {
    if (!p || !n) return ja_fail(JA_ERR_INVALID_ARG, "null argument");
    *n = count_memberships(*p);
    return JA_OK;
}
extern "C" ja_status_t ja_exprog_bind(ja_exprog_t* p, int64_t index) {
    if (!p) return ja_fail(JA_ERR_INVALID_ARG, "null program");
    if (count_memberships(*p) > MEMBERSHIP_LIST_LIMIT)
        return ja_fail(JA_ERR_UNSUPPORTED, "more than %lld memberships: bind the partitions with ja_exprog_bind_members or let ja_exprog_place choose",
                       (long long)MEMBERSHIP_LIST_LIMIT);
    std::vector<std::vector<std::vector<int>>> all;
    enumerate_memberships(*p, &all);
    if (index < 0 || index >= (int64_t)all.size()) return ja_fail(JA_ERR_INVALID_ARG, "membership %lld of %lld", (long long)index, (long long)all.size());
    bind_membership(p, all[index]);
    return check_static(*p);
}
extern "C" ja_status_t ja_exprog_membership(const ja_exprog_t* p, const char* partition, uint64_t* members) {
    if (!p || !partition || !members) return ja_fail(JA_ERR_INVALID_ARG, "null argument");
    const int k = find_part(*p, partition);
    if (k < 0) return ja_fail(JA_ERR_INVALID_ARG, "no partition '%s'", partition);
    if (!p->parts[k].bound) return ja_fail(JA_ERR_INVALID_ARG, "partition '%s' has no members yet", partition);
    *members = 0;
    for (int s : p->parts[k].members) *members |= 1ull << s;
    return JA_OK;
}

extern "C" ja_status_t ja_exprog_closure(const ja_exprog_t* p, int64_t* n, uint64_t* aggregate, int32_t* site) {
    ja_status_t s = need_bound(p);
    if (s != JA_OK) return s;
    std::vector<Flat> acts;
    expand(*p, &acts);
    const State st = closure_of(*p, acts);
    if (n) *n = (int64_t)st.size();
    int64_t i = 0;
    for (const auto& e : st) {
        if (aggregate) aggregate[i] = e.second;
        if (site) site[i] = e.first;
        ++i;
    }
    return JA_OK;
}
extern "C" ja_status_t ja_exprog_check(const ja_exprog_t* p, int32_t* well_formed, int32_t* valid) {
    ja_status_t s = need_bound(p);
    if (s != JA_OK) return s;
    bool wf, v;
    check_bound(*p, &wf, &v);
    if (well_formed) *well_formed = wf;
    if (valid) *valid = v;
    return JA_OK;
}
extern "C" ja_status_t ja_exprog_valid_any(const ja_exprog_t* p, int32_t* valid) {
    if (!p || !valid) return ja_fail(JA_ERR_INVALID_ARG, "null argument");
    if (count_memberships(*p) > MEMBERSHIP_LIST_LIMIT)
        return ja_fail(JA_ERR_UNSUPPORTED, "more than %lld memberships to try", (long long)MEMBERSHIP_LIST_LIMIT);
    std::vector<std::vector<std::vector<int>>> all;
    enumerate_memberships(*p, &all);
    *valid = 0;
    for (const auto& mem : all) {
        Prog q = *p;
        bind_membership(&q, mem);
        if (valid_bound(q)) {
            *valid = 1;
            break;
        }
    }
    return JA_OK;
}

extern "C" ja_status_t ja_exprog_simulate(const ja_exprog_t* p, const ja_machine_t* machine, double* completion_ms,
                                          double* start_ms, double* aggregated_ms, double* finish_ms) {
    ja_status_t s = need_bound(p);
    if (s != JA_OK) return s;
    if ((s = check_machine(machine, *p)) != JA_OK) return s;
    double ms = 0;
    if (!simulate(*p, *machine, &ms, start_ms, aggregated_ms, finish_ms))
        return ja_fail(JA_ERR_INVALID_ARG, "the program is not well-formed: an action never becomes enabled");
    if (completion_ms) *completion_ms = ms;
    return JA_OK;
}

extern "C" ja_status_t ja_exprog_body(ja_exprog_t* p, int32_t body) {
    ja_status_t s = need_bound(p);
    if (s != JA_OK) return s;
    if (body == JA_BODY_NAIVE) naive_body(p);
    else if (body == JA_BODY_BUTTERFLY) butterfly_body(p);
    else if (body != JA_BODY_OWN) return ja_fail(JA_ERR_INVALID_ARG, "body %d", body);
    return JA_OK;
}
extern "C" ja_status_t ja_exprog_normalise(ja_exprog_t* p) {
    ja_status_t s = need_bound(p);
    if (s != JA_OK) return s;
    normalise(p);
    return JA_OK;
}
extern "C" ja_status_t ja_exprog_rewrite(ja_exprog_t* p, int32_t rule, int32_t i, int32_t j, uint64_t a, uint64_t b, int32_t* applied) {
    ja_status_t s = need_bound(p);
    if (s != JA_OK) return s;
    if (!applied) return ja_fail(JA_ERR_INVALID_ARG, "null argument");
    if (!is_normal(*p)) return ja_fail(JA_ERR_INVALID_ARG, "the rules work on a normalised program (ja_exprog_normalise)");
    if (rule < JA_RULE_INSERT || rule > JA_RULE_SOURCE) return ja_fail(JA_ERR_INVALID_ARG, "rule %d", rule);
    Prog q;
    *applied = rewrite(*p, rule, i, j, a, b, &q) ? 1 : 0;
    if (*applied) *p = q;
    return JA_OK;
}
extern "C" ja_status_t ja_exprog_synthesize(ja_exprog_t* p, const ja_machine_t* machine, int32_t depth, int32_t beam, double* ms) {
    ja_status_t s = need_bound(p);
    if (s != JA_OK) return s;
    if ((s = check_machine(machine, *p)) != JA_OK) return s;
    if (depth < 0 || beam < 1) return ja_fail(JA_ERR_INVALID_ARG, "depth >= 0 and beam >= 1");
    Prog start;
    double t0 = 0;
    if (!p->actions.empty()) {
        start = *p;
        normalise(&start);
        if (!valid_bound(start) || !simulate(start, *machine, &t0, nullptr, nullptr, nullptr))
            return ja_fail(JA_ERR_INVALID_ARG, "the program's own body is not valid");
    } else {
        if (!best_constructed(*p, *machine, JA_BODY_BEST, &start, &t0)) return ja_fail(JA_ERR_INVALID_ARG, "OUT cannot be satisfied");
        normalise(&start);
    }
    std::pair<double, Prog> best(t0, start);
    std::vector<std::pair<double, Prog>> level(1, best);
    std::set<Key> seen;
    seen.insert(key_of(start));
    std::vector<Prog> nb;
    for (int d = 0; d < depth; ++d) {
        std::vector<std::pair<double, Prog>> nxt;
        for (const auto& cur : level) {
            neighbours(cur.second, &nb);
            for (const Prog& r : nb) {
                if (!seen.insert(key_of(r)).second) continue;
                double t;
                if (!simulate(r, *machine, &t, nullptr, nullptr, nullptr)) continue;
                nxt.push_back({t, r});
            }
        }
        if (nxt.empty()) break;
        std::stable_sort(nxt.begin(), nxt.end(), [](const std::pair<double, Prog>& x, const std::pair<double, Prog>& y) {
            return x.first != y.first ? x.first < y.first : x.second.actions.size() < y.second.actions.size();
        });
        if ((int)nxt.size() > beam) nxt.resize(beam);
        level.swap(nxt);
        if (level[0].first < best.first * (1.0 - 1e-12)) best = level[0];
    }
    *p = best.second;
    if (ms) *ms = best.first;
    return JA_OK;
}
extern "C" ja_status_t ja_exprog_place(ja_exprog_t* p, const ja_machine_t* machine, int32_t body, double* ms) {
    if (!p) return ja_fail(JA_ERR_INVALID_ARG, "null program");
    ja_status_t s = check_machine(machine, *p);
    if (s != JA_OK) return s;
    if (body < JA_BODY_OWN || body > JA_BODY_BEST) return ja_fail(JA_ERR_INVALID_ARG, "body %d", body);
    bool found = false;
    Prog best;
    double best_ms = 0, best_gb = 0;
    if (count_memberships(*p) <= PLACE_ENUMERATION_LIMIT) {
        std::vector<std::vector<std::vector<int>>> all;
        enumerate_memberships(*p, &all);
        for (const auto& mem : all) {
            Prog q = *p;
            bind_membership(&q, mem);
            Prog c;
            double t;
            if (!best_constructed(q, *machine, body, &c, &t)) continue;
            const double gb = bytes_sent(c);
            if (better_placement(t, gb, found, best_ms, best_gb)) {
                best = c;
                best_ms = t;
                best_gb = gb;
                found = true;
            }
        }
    } else {
        // steepest descent over exchanges of two sites between partitions, from the first membership in enumeration order
        // (the free sites dealt to the size-declared partitions in ascending order)
        std::vector<int> unbound;
        std::set<int> taken;
        for (size_t i = 0; i < p->parts.size(); ++i) {
            if (p->parts[i].bound) taken.insert(p->parts[i].members.begin(), p->parts[i].members.end());
            else unbound.push_back((int)i);
        }
        std::vector<std::vector<int>> cur;
        {
            std::vector<int> free_sites;
            for (int g : p->gpus)
                if (!taken.count(g)) free_sites.push_back(g);
            size_t at = 0;
            for (int k : unbound) {
                cur.push_back(std::vector<int>(free_sites.begin() + at, free_sites.begin() + at + p->parts[k].size));
                at += p->parts[k].size;
            }
        }
        auto cost_of = [&](const std::vector<std::vector<int>>& mem, Prog* c, double* t) {
            Prog q = *p;
            bind_membership(&q, mem);
            return best_constructed(q, *machine, body, c, t);
        };
        found = cost_of(cur, &best, &best_ms);
        if (found) best_gb = bytes_sent(best);
        bool improved = true;
        while (improved) {
            improved = false;
            std::vector<std::vector<int>> pick;
            Prog pick_prog;
            double pick_ms = 0, pick_gb = 0;
            bool any = false;
            for (size_t a = 0; a < cur.size(); ++a)
                for (size_t b = a + 1; b < cur.size(); ++b)
                    for (size_t i = 0; i < cur[a].size(); ++i)
                        for (size_t j = 0; j < cur[b].size(); ++j) {
                            std::vector<std::vector<int>> nxt = cur;
                            std::swap(nxt[a][i], nxt[b][j]);
                            Prog c;
                            double t;
                            if (!cost_of(nxt, &c, &t)) continue;
                            const double gb = bytes_sent(c);
                            if (any ? better_placement(t, gb, true, pick_ms, pick_gb) : better_placement(t, gb, found, best_ms, best_gb)) {
                                pick = nxt;
                                pick_prog = c;
                                pick_ms = t;
                                pick_gb = gb;
                                any = true;
                            }
                        }
            if (any) {
                cur = pick;
                best = pick_prog;
                best_ms = pick_ms;
                best_gb = pick_gb;
                found = true;
                improved = true;
            }
        }
    }
    if (!found) return ja_fail(JA_ERR_INVALID_ARG, "no membership makes the program valid");
    *p = best;
    if (ms) *ms = best_ms;
    return JA_OK;
}

extern "C" ja_status_t ja_exprog_bind_members(ja_exprog_t* p, const char* partition, const int32_t* sites, int32_t n) {
    if (!p || !partition || !sites) return ja_fail(JA_ERR_INVALID_ARG, "null argument");
    const int k = find_part(*p, partition);
    if (k < 0) return ja_fail(JA_ERR_INVALID_ARG, "no partition '%s'", partition);
    if (p->parts[k].bound) return ja_fail(JA_ERR_INVALID_ARG, "partition '%s' already has members", partition);
    if (n != p->parts[k].size) return ja_fail(JA_ERR_INVALID_ARG, "partition '%s' has size %d", partition, p->parts[k].size);
    Prog q = *p;
    q.parts[k].members.assign(sites, sites + n);
    std::sort(q.parts[k].members.begin(), q.parts[k].members.end());
    q.parts[k].bound = true;
    ja_status_t st = check_static(q);
    if (st != JA_OK) return st;
    *p = q;
    return JA_OK;
}

namespace {

// the overlay of a producer's and a consumer's tiling of one tensor and the preamble built on it (Section 5.3)
struct OverlayCell {
    int64_t j, pb, cb;                 // atom number (row-major over the overlay), flat producer block, flat consumer block
    int64_t lo[8], hi[8];              // its box
    double gb;
};
struct Overlay {
    int rank = 0;
    std::vector<std::vector<int64_t>> ps, cs, ov;
    std::vector<OverlayCell> cells;
    std::vector<std::pair<int64_t, int>> atom_jc;   // per ExProg atom (declaration order): (atom number, copy)
};

ja_status_t make_preamble(int rank, const std::vector<std::vector<int64_t>>& ps, const std::vector<std::vector<int64_t>>& cs,
                          int m, const int32_t* copy_site, const int32_t* consumer_specs, int n_specs, int width_bytes,
                          Prog* p, Overlay* o) {
    o->rank = rank;
    o->ps = ps;
    o->cs = cs;
    o->ov.assign(rank, {});
    int64_t n_pblocks = 1, n_cblocks = 1, n_cells = 1;
    for (int d = 0; d < rank; ++d) {
        if (ps[d].size() < 2 || cs[d].size() < 2) return ja_fail(JA_ERR_TILING, "index %d: at least two split points", d);
        for (const auto* v : {&ps[d], &cs[d]}) {
            if ((*v)[0] != 0) return ja_fail(JA_ERR_TILING, "index %d: split points start at 0", d);
            for (size_t i = 1; i < v->size(); ++i)
                if ((*v)[i] <= (*v)[i - 1]) return ja_fail(JA_ERR_TILING, "index %d: split points must increase", d);
        }
        if (ps[d].back() != cs[d].back()) return ja_fail(JA_ERR_SHAPE, "index %d: the two tilings differ in extent", d);
        std::set<int64_t> u(ps[d].begin(), ps[d].end());
        u.insert(cs[d].begin(), cs[d].end());
        o->ov[d].assign(u.begin(), u.end());
        n_pblocks *= (int64_t)ps[d].size() - 1;
        n_cblocks *= (int64_t)cs[d].size() - 1;
        n_cells *= (int64_t)o->ov[d].size() - 1;
    }
    if (n_cells * m > 64) return ja_fail(JA_ERR_INVALID_ARG, "%lld atoms x %d copies: at most 64 ExProg atoms", (long long)n_cells, m);
    std::set<int> g;
    for (int64_t i = 0; i < n_pblocks * m; ++i) g.insert(copy_site[i]);
    for (int i = 0; i < n_specs; ++i) g.insert(i);
    p->gpus.assign(g.begin(), g.end());
    for (int i = 0; i < n_specs; ++i) {
        if (consumer_specs[i] < 0 || consumer_specs[i] >= n_cblocks)
            return ja_fail(JA_ERR_INVALID_ARG, "function spec %d names block %d of %lld", i, consumer_specs[i], (long long)n_cblocks);
        ExPartition q;
        q.name = "S" + std::to_string(i + 1);
        q.size = 1;
        p->parts.push_back(q);
    }
    auto owner = [](const std::vector<int64_t>& s, int64_t lo) {
        int i = 0;
        while (!(s[i] <= lo && lo < s[i + 1])) ++i;
        return i;
    };
    std::vector<int> c(rank, 0);
    for (int64_t j = 0; j < n_cells; ++j) {
        OverlayCell ce;
        ce.j = j;
        ce.pb = ce.cb = 0;
        int64_t card = 1;
        for (int d = 0; d < rank; ++d) {
            ce.lo[d] = o->ov[d][c[d]];
            ce.hi[d] = o->ov[d][c[d] + 1];
            card *= ce.hi[d] - ce.lo[d];
            ce.pb = ce.pb * ((int64_t)ps[d].size() - 1) + owner(ps[d], ce.lo[d]);
            ce.cb = ce.cb * ((int64_t)cs[d].size() - 1) + owner(cs[d], ce.lo[d]);
        }
        ce.gb = (double)(card * width_bytes) / 1e9;
        o->cells.push_back(ce);
        for (int d = rank - 1; d >= 0; --d) {
            if (++c[d] < (int)o->ov[d].size() - 1) break;
            c[d] = 0;
        }
    }
    // IN: by site, then atom, then copy
    std::vector<std::tuple<int, int64_t, int, double>> entries;
    for (const OverlayCell& ce : o->cells)
        for (int k = 0; k < m; ++k) entries.push_back(std::make_tuple(copy_site[ce.pb * m + k], ce.j, k, ce.gb));
    std::sort(entries.begin(), entries.end());
    std::map<std::pair<int64_t, int>, int> index;
    for (const auto& e : entries) {
        ExAtom a;
        a.name = "a" + std::to_string(std::get<1>(e)) + "_" + std::to_string(std::get<2>(e));
        a.site = std::get<0>(e);
        a.gb = std::get<3>(e);
        index[{std::get<1>(e), std::get<2>(e)}] = (int)p->atoms.size();
        o->atom_jc.push_back({std::get<1>(e), std::get<2>(e)});
        p->atoms.push_back(a);
    }
    for (const OverlayCell& ce : o->cells) {
        uint64_t x = 0;
        for (int k = 0; k < m; ++k) x |= 1ull << index[{ce.j, k}];
        for (int i = 0; i < n_specs; ++i)
            if (consumer_specs[i] == ce.cb) {
                ExTarget t;
                t.part = i;
                p->out.push_back({x, t});
            }
    }
    if ((int)p->gpus.size() != n_specs)
        return ja_fail(JA_ERR_INVALID_ARG, "one function spec of op per GPU: the partitions of size one must cover the GPUs");
    return check_static(*p);
}

}  // namespace

extern "C" ja_status_t ja_exprog_preamble(int32_t rank, const int64_t* producer_splits, const int32_t* n_producer_splits,
                                          const int64_t* consumer_splits, const int32_t* n_consumer_splits, int32_t m,
                                          const int32_t* copy_site, const int32_t* consumer_specs, int32_t n_specs,
                                          int32_t width_bytes, ja_exprog_t** out) {
    if (rank < 1 || rank > 8 || !producer_splits || !n_producer_splits || !consumer_splits || !n_consumer_splits || m < 1 ||
        !copy_site || !consumer_specs || n_specs < 1 || width_bytes < 1 || !out)
        return ja_fail(JA_ERR_INVALID_ARG, "bad argument");
    std::vector<std::vector<int64_t>> ps(rank), cs(rank);
    const int64_t *pp = producer_splits, *cp = consumer_splits;
    for (int d = 0; d < rank; ++d) {
        if (n_producer_splits[d] < 2 || n_consumer_splits[d] < 2) return ja_fail(JA_ERR_TILING, "index %d: at least two split points", d);
        ps[d].assign(pp, pp + n_producer_splits[d]);
        cs[d].assign(cp, cp + n_consumer_splits[d]);
        pp += n_producer_splits[d];
        cp += n_consumer_splits[d];
    }
    Prog* p = new Prog();
    Overlay o;
    ja_status_t st = make_preamble(rank, ps, cs, m, copy_site, consumer_specs, n_specs, width_bytes, p, &o);
    if (st != JA_OK) {
        delete p;
        return st;
    }
    *out = p;
    return JA_OK;
}

namespace {
// A firing order of a bound program and the parts of every aggregation: repeated passes over the expanded actions in body
// order; an action fires the first time aggregates at its source partition its aggregate (the partition with the fewest parts,
// candidates in ascending order of their masks, so the parts come out in ascending order of their first atoms). Actions that
// never become enabled are left out (the program is then not well-formed).
struct Fired {
    int act;
    std::vector<uint64_t> parts;
};
void firing_order(const Prog& p, const std::vector<Flat>& acts, std::vector<Fired>* order) {
    order->clear();
    std::map<int, std::set<uint64_t>> have;
    for (size_t i = 0; i < p.atoms.size(); ++i) have[p.atoms[i].site].insert(1ull << i);
    std::vector<bool> fired(acts.size(), false);
    bool progress = true;
    while (progress) {
        progress = false;
        for (size_t i = 0; i < acts.size(); ++i) {
            if (fired[i]) continue;
            CoverParts cp;
            for (uint64_t y : have[acts[i].site])
                if ((y & ~acts[i].agg) == 0) cp.cands.push_back(y);
            cp.rec(acts[i].agg);
            if (cp.best.empty()) continue;
            fired[i] = true;
            progress = true;
            order->push_back({(int)i, cp.best});
            have[acts[i].site].insert(acts[i].agg);
            for (int d : acts[i].dests) have[d].insert(acts[i].agg);
        }
    }
}
}  // namespace

extern "C" ja_status_t ja_exprog_schedule(const ja_exprog_t* p, int32_t* n_fired, int32_t* n_parts_total, int32_t* action,
                                          int32_t* part_begin, uint64_t* parts) {
    ja_status_t st = need_bound(p);
    if (st != JA_OK) return st;
    std::vector<Flat> acts;
    expand(*p, &acts);
    std::vector<Fired> order;
    firing_order(*p, acts, &order);
    if (order.size() != acts.size()) return ja_fail(JA_ERR_INVALID_ARG, "the program is not well-formed: an action never becomes enabled");
    int32_t total = 0;
    for (size_t i = 0; i < order.size(); ++i) {
        if (action) action[i] = order[i].act;
        if (part_begin) part_begin[i] = total;
        for (uint64_t y : order[i].parts) {
            if (parts) parts[total] = y;
            ++total;
        }
    }
    if (part_begin) part_begin[order.size()] = total;
    if (n_fired) *n_fired = (int32_t)order.size();
    if (n_parts_total) *n_parts_total = total;
    return JA_OK;
}

extern "C" ja_status_t ja_exchange_combine(const void* const* parts, int32_t n_parts, void* out, int64_t bytes, ja_dtype_t dtype,
                                           ja_agg_t agg, void* cuda_stream) {
    if (!parts || !out || bytes < 1) return ja_fail(JA_ERR_INVALID_ARG, "null argument");
    if (agg != JA_AGG_SUM && agg != JA_AGG_MAX) return ja_fail(JA_ERR_INVALID_ARG, "SUM or MAX");
    if (dtype != JA_F32 && dtype != JA_BF16 && dtype != JA_F16) return ja_fail(JA_ERR_DTYPE, "unknown cell type");
    if (bytes % 16) return ja_fail(JA_ERR_ALIGNMENT, "the buffers are read and written in 16-byte accesses: %lld bytes is not a whole number of them", (long long)bytes);
    if ((uintptr_t)out % 16) return ja_fail(JA_ERR_ALIGNMENT, "out must be 16-byte aligned");
    for (int i = 0; i < n_parts; ++i)
        if (!parts[i] || (uintptr_t)parts[i] % 16) return ja_fail(JA_ERR_ALIGNMENT, "part %d must be a 16-byte aligned device pointer", i);
    return ja_launch_exchange_combine(parts, n_parts, out, bytes, dtype, agg, (cudaStream_t)cuda_stream);
}

// Scratch of ja_exchange_execute: a stream-ordered pool of the library's own per device that keeps what it has been given
// (the default pool hands memory back to the driver at every synchronisation, and getting a gigabyte again costs milliseconds);
// ja_exchange_trim returns it.
namespace {
std::mutex g_pool_mu;
std::map<int, cudaMemPool_t> g_pools;
ja_status_t exchange_pool(cudaMemPool_t* out) {
    int dev = 0;
    JA_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lk(g_pool_mu);
    auto it = g_pools.find(dev);
    if (it == g_pools.end()) {
        cudaMemPoolProps props;
        memset(&props, 0, sizeof props);
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = dev;
        cudaMemPool_t mp = nullptr;
        JA_CUDA(cudaMemPoolCreate(&mp, &props));
        uint64_t keep = UINT64_MAX;
        JA_CUDA(cudaMemPoolSetAttribute(mp, cudaMemPoolAttrReleaseThreshold, &keep));
        it = g_pools.insert({dev, mp}).first;
    }
    *out = it->second;
    return JA_OK;
}
}  // namespace

extern "C" ja_status_t ja_exchange_trim(void) {
    std::lock_guard<std::mutex> lk(g_pool_mu);
    for (auto& kv : g_pools) JA_CUDA(cudaMemPoolTrimTo(kv.second, 0));
    return JA_OK;
}

// ---------------------------------------------------------------------------------- execution on one GPU (Section 5.3)
// The sites of the program are regions of this GPU's memory; a transfer is a device-to-device copy (on a machine with
// several GPUs it would be a peer copy), a local aggregation one launch of the combine kernel, decompose and recompose
// one batched box-copy launch each. Actions are issued on one stream in a firing order of the program.
namespace {

// Everything ja_exchange_execute and an exchange plan need beyond the relations' payloads, worked out on the host.
struct ExBuffer {
    int site;
    uint64_t agg;
    int64_t off, bytes;
    int producer_site;      // whose stream writes it: -1 = decompose (before the sites' streams fork)
};
struct ExStep {
    int site;
    int out;                        // buffer of the aggregate at the source
    std::vector<int> parts;         // >= 2: a local aggregation into `out`; 1: `out` is already materialised
    std::vector<int> dests;         // buffers the aggregate is transferred to
};
struct ExBuild {
    std::vector<ExBuffer> bufs;
    std::vector<ExStep> steps;
    std::vector<JaBoxCopy> boxes;   // n_in decompose boxes (box a fills buffer a, the atoms come first), then n_out recompose boxes
    std::vector<int> out_box_buf;   // the buffer every recompose box reads
    int n_in = 0, n_out = 0;
    bool vec_in = true, vec_out = true;
    int64_t max_in = 0, max_out = 0, scratch = 0, table_off = 0, table_bytes = 0;
    int64_t n_aggregations = 0, n_transfers = 0, transfer_bytes = 0, aggregation_bytes = 0;
    std::vector<int> sites;         // the sites that run a step
    ja_dtype_t dtype = JA_BF16;
    int esize = 2;
    ja_agg_t agg = JA_AGG_SUM;
    const char* src_base = nullptr;
    char* dst_base = nullptr;
};

ja_status_t build_exchange(const ja_exprog_t* prog, const ja_relation_t* partials, const int32_t* copy_site, const int32_t* consumer_specs,
                           int32_t n_specs, ja_agg_t agg, ja_relation_t* dst, ExBuild* B) {
    ja_status_t st = need_bound(prog);
    if (st != JA_OK) return st;
    if (!partials || !dst || !copy_site || !consumer_specs || n_specs < 1) return ja_fail(JA_ERR_INVALID_ARG, "null argument");
    const int rank = dst->rank;
    if (partials->rank != rank + 1) return ja_fail(JA_ERR_SHAPE, "a partial relation has the copy index in front: rank %d expected, got %d", rank + 1, partials->rank);
    if (partials->nblk[0] != partials->extent[0]) return ja_fail(JA_ERR_TILING, "the copy index of a partial relation must be cut into unit intervals");
    for (int d = 0; d < rank; ++d)
        if (partials->extent[d + 1] != dst->extent[d]) return ja_fail(JA_ERR_SHAPE, "extent of dimension %d differs", d);
    if (partials->dtype != dst->dtype) return ja_fail(JA_ERR_DTYPE, "the exchange moves and aggregates atoms in the partial relation's cell type: the consumer relation must have it too");
    if (partials->base == dst->base) return ja_fail(JA_ERR_INVALID_ARG, "the consumer relation aliases the partial relation");
    if (rank > 3) return ja_fail(JA_ERR_UNSUPPORTED, "tensors of rank above 3");
    const int m = (int)partials->extent[0];
    if (agg != JA_AGG_SUM && agg != JA_AGG_MAX && !(agg == JA_AGG_NONE && m == 1))
        return ja_fail(JA_ERR_INVALID_ARG, "%d copies of every atom need SUM or MAX aggregation", m);
    // the preamble these relations generate must be the program's
    std::vector<std::vector<int64_t>> ps(rank), cs(rank);
    for (int d = 0; d < rank; ++d) {
        ps[d] = partials->splits[d + 1];
        cs[d] = dst->splits[d];
    }
    Prog pre;
    Overlay ov;
    if ((st = make_preamble(rank, ps, cs, m, copy_site, consumer_specs, n_specs, partials->esize, &pre, &ov)) != JA_OK) return st;
    bool same = pre.gpus == prog->gpus && pre.atoms.size() == prog->atoms.size() && pre.out.size() == prog->out.size() &&
                pre.parts.size() == prog->parts.size();
    for (size_t i = 0; same && i < pre.atoms.size(); ++i)
        same = pre.atoms[i].name == prog->atoms[i].name && pre.atoms[i].site == prog->atoms[i].site && pre.atoms[i].gb == prog->atoms[i].gb;
    for (size_t i = 0; same && i < pre.out.size(); ++i) same = pre.out[i].first == prog->out[i].first && pre.out[i].second == prog->out[i].second;
    for (size_t i = 0; same && i < pre.parts.size(); ++i) same = pre.parts[i].name == prog->parts[i].name && prog->parts[i].members.size() == 1;
    if (!same) return ja_fail(JA_ERR_INVALID_ARG, "the program's preamble is not the one these relations, copy sites and function specs generate");
    if (!valid_bound(*prog)) return ja_fail(JA_ERR_INVALID_ARG, "the program is not valid (Definition \"Closure; validity\")");

    B->dtype = partials->dtype;
    B->esize = partials->esize;
    B->agg = agg;
    B->src_base = (const char*)partials->base;
    B->dst_base = (char*)dst->base;
    // firing order and the parts of every aggregation
    std::vector<Flat> acts;
    expand(*prog, &acts);
    std::vector<Fired> order;
    firing_order(*prog, acts, &order);
    // buffers: one per (aggregate, site) materialisation
    auto atom_bytes = [&](uint64_t agg_mask) {
        const int a = __builtin_ctzll(agg_mask);
        const OverlayCell& ce = ov.cells[ov.atom_jc[a].first];
        int64_t cells = 1;
        for (int d = 0; d < rank; ++d) cells *= ce.hi[d] - ce.lo[d];
        return cells * (int64_t)partials->esize;
    };
    std::map<std::pair<int, uint64_t>, int> index;
    auto buffer = [&](int site, uint64_t x, int producer_site) {
        auto key = std::make_pair(site, x);
        auto it = index.find(key);
        if (it != index.end()) return it->second;
        B->bufs.push_back({site, x, B->scratch, atom_bytes(x), producer_site});
        B->scratch += (atom_bytes(x) + 255) / 256 * 256;
        index[key] = (int)B->bufs.size() - 1;
        return (int)B->bufs.size() - 1;
    };
    for (size_t a = 0; a < prog->atoms.size(); ++a) buffer(prog->atoms[a].site, 1ull << a, -1);
    std::set<int> step_sites;
    for (const Fired& f : order) {
        const Flat& a = acts[f.act];
        if (f.parts.size() > JA_EXCHANGE_MAX_PARTS)
            return ja_fail(JA_ERR_UNSUPPORTED, "an aggregation of %d parts (at most %d)", (int)f.parts.size(), JA_EXCHANGE_MAX_PARTS);
        ExStep stp;
        stp.site = a.site;
        for (uint64_t y : f.parts) stp.parts.push_back(index.at({a.site, y}));
        stp.out = buffer(a.site, a.agg, a.site);
        if (f.parts.size() >= 2) {
            ++B->n_aggregations;
            B->aggregation_bytes += ((int64_t)f.parts.size() + 1) * atom_bytes(a.agg);
        }
        for (int d : a.dests) {
            const bool fresh = !index.count({d, a.agg});
            const int b = buffer(d, a.agg, a.site);
            if (fresh && b != stp.out) {               // a second delivery of an aggregate that is already there moves nothing
                stp.dests.push_back(b);
                ++B->n_transfers;
                B->transfer_bytes += atom_bytes(a.agg);
            }
        }
        if (f.parts.size() >= 2 || !stp.dests.empty()) {
            step_sites.insert(a.site);
            B->steps.push_back(stp);
        }
    }
    B->sites.assign(step_sites.begin(), step_sites.end());
    // decompose and recompose tables
    const int64_t ntrail = partials->nblocks / m;
    auto box_of = [&](const OverlayCell& ce, const std::vector<std::vector<int64_t>>& tiling, int64_t blk, int64_t blk_off, bool from_block, int64_t buf_off) {
        // the block's extents and the box's offset inside it, padded to three dimensions in front
        int64_t bext[3] = {1, 1, 1}, off[3] = {0, 0, 0}, n[3] = {1, 1, 1};
        int64_t rem = blk;
        for (int d = rank - 1; d >= 0; --d) {
            const int64_t nb = (int64_t)tiling[d].size() - 1, k = rem % nb;
            rem /= nb;
            bext[3 - rank + d] = tiling[d][k + 1] - tiling[d][k];
            off[3 - rank + d] = ce.lo[d] - tiling[d][k];
            n[3 - rank + d] = ce.hi[d] - ce.lo[d];
        }
        const int64_t es = partials->esize;
        JaBoxCopy b;
        b.n0 = n[0];
        b.n1 = n[1];
        b.run_bytes = n[2] * es;
        const int64_t blk_pitch1 = bext[2] * es, blk_pitch0 = bext[1] * blk_pitch1;
        const int64_t in_blk = blk_off + off[0] * blk_pitch0 + off[1] * blk_pitch1 + off[2] * es;
        const int64_t dense1 = n[2] * es, dense0 = n[1] * dense1;
        if (from_block) {
            b.src_off = in_blk; b.src_pitch0 = blk_pitch0; b.src_pitch1 = blk_pitch1;
            b.dst_off = buf_off; b.dst_pitch0 = dense0; b.dst_pitch1 = dense1;
        } else {
            b.dst_off = in_blk; b.dst_pitch0 = blk_pitch0; b.dst_pitch1 = blk_pitch1;
            b.src_off = buf_off; b.src_pitch0 = dense0; b.src_pitch1 = dense1;
        }
        return b;
    };
    auto aligned16 = [](const JaBoxCopy& b) {
        return ((b.src_off | b.dst_off | b.src_pitch0 | b.src_pitch1 | b.dst_pitch0 | b.dst_pitch1 | b.run_bytes) & 15) == 0;
    };
    for (size_t a = 0; a < prog->atoms.size(); ++a) {
        const OverlayCell& ce = ov.cells[ov.atom_jc[a].first];
        const int c = ov.atom_jc[a].second;
        const JaBoxCopy b = box_of(ce, ps, ce.pb, partials->blk_off[c * ntrail + ce.pb], true, B->bufs[index.at({prog->atoms[a].site, 1ull << a})].off);
        B->vec_in = B->vec_in && aligned16(b);
        B->max_in = std::max(B->max_in, b.n0 * b.n1 * b.run_bytes);
        B->boxes.push_back(b);
    }
    B->n_in = (int)B->boxes.size();
    std::set<int64_t> done;
    for (int i = 0; i < n_specs; ++i) {
        const int site = prog->parts[i].members[0];
        for (const OverlayCell& ce : ov.cells) {
            if (ce.cb != consumer_specs[i] || done.count(ce.j)) continue;
            done.insert(ce.j);
            uint64_t x = 0;
            for (size_t a = 0; a < prog->atoms.size(); ++a)
                if (ov.atom_jc[a].first == ce.j) x |= 1ull << a;
            auto it = index.find({site, x});
            if (it == index.end()) return ja_fail(JA_ERR_INVALID_ARG, "internal: a required aggregate was never materialised");
            const JaBoxCopy b = box_of(ce, cs, ce.cb, dst->blk_off[ce.cb], false, B->bufs[it->second].off);
            B->vec_out = B->vec_out && aligned16(b);
            B->max_out = std::max(B->max_out, b.n0 * b.n1 * b.run_bytes);
            B->boxes.push_back(b);
            B->out_box_buf.push_back(it->second);
        }
    }
    B->n_out = (int)B->boxes.size() - B->n_in;
    B->table_bytes = (int64_t)B->boxes.size() * (int64_t)sizeof(JaBoxCopy);
    B->table_off = B->scratch;
    B->scratch += (B->table_bytes + 255) / 256 * 256;
    return JA_OK;
}

void fill_stats(const ExBuild& B, int64_t* stats) {
    if (!stats) return;
    stats[0] = B.n_aggregations;
    stats[1] = B.n_transfers;
    stats[2] = B.transfer_bytes;
    stats[3] = B.scratch;
    stats[4] = B.aggregation_bytes;
}

// one step on `stream`: the local aggregation, then the transfers
ja_status_t issue_step(const ExBuild& B, const ExStep& s, char* pool, cudaStream_t stream) {
    char* here = pool + B.bufs[s.out].off;
    if (s.parts.size() >= 2) {
        const void* parts[JA_EXCHANGE_MAX_PARTS];
        for (size_t k = 0; k < s.parts.size(); ++k) parts[k] = pool + B.bufs[s.parts[k]].off;
        ja_status_t rc = ja_launch_exchange_combine(parts, (int)s.parts.size(), here, B.bufs[s.out].bytes, B.dtype, B.agg, stream);
        if (rc != JA_OK) return rc;
    }
    for (int d : s.dests)
        if (cudaMemcpyAsync(pool + B.bufs[d].off, here, (size_t)B.bufs[s.out].bytes, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
            return ja_fail(JA_ERR_CUDA, "a transfer failed");
    return JA_OK;
}

}  // namespace

extern "C" ja_status_t ja_exchange_execute(const ja_exprog_t* prog, const ja_relation_t* partials, const int32_t* copy_site,
                                           const int32_t* consumer_specs, int32_t n_specs, ja_agg_t agg, ja_relation_t* dst,
                                           int64_t* stats, void* cuda_stream) {
    ExBuild B;
    ja_status_t st = build_exchange(prog, partials, copy_site, consumer_specs, n_specs, agg, dst, &B);
    if (st != JA_OK) return st;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        JA_CUDA(cudaStreamIsCapturing(stream, &cap));
        if (cap != cudaStreamCaptureStatusNone)
            return ja_fail(JA_ERR_UNSUPPORTED, "ja_exchange_execute was called on a stream that is being captured: its box tables are staged from "
                                               "host memory of this call, which a replay would read too late (an exchange plan can be captured)");
    }
    char* pool = nullptr;
    cudaMemPool_t mp = nullptr;
    if ((st = exchange_pool(&mp)) != JA_OK) return st;
    JA_CUDA(cudaMallocFromPoolAsync((void**)&pool, (size_t)B.scratch, mp, stream));
    ja_status_t rc = JA_OK;
    do {
        if (cudaMemcpyAsync(pool + B.table_off, B.boxes.data(), (size_t)B.table_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) {
            rc = ja_fail(JA_ERR_CUDA, "copying the box tables failed");
            break;
        }
        const JaBoxCopy* d_boxes = (const JaBoxCopy*)(pool + B.table_off);
        if ((rc = ja_launch_box_copies(B.src_base, pool, d_boxes, B.n_in, B.max_in, B.vec_in, B.esize, stream)) != JA_OK) break;
        for (const ExStep& s : B.steps)
            if ((rc = issue_step(B, s, pool, stream)) != JA_OK) break;
        if (rc != JA_OK) break;
        rc = ja_launch_box_copies(pool, B.dst_base, d_boxes + B.n_in, B.n_out, B.max_out, B.vec_out, B.esize, stream);
    } while (false);
    cudaFreeAsync(pool, stream);
    if (rc != JA_OK) return rc;
    fill_stats(B, stats);
    return JA_OK;
}

// ---- an exchange plan: the same program with its buffers and tables kept on the device, issued as dataflow ------------------
// Every site that runs a step has a stream of its own; a step waits for the buffers other sites' streams write (events), so what
// a capture of ja_exchange_plan_run records is the program's dependency graph -- kernels and copies as vertices -- and actions of
// different sites may run at the same time, copies on the copy engines beside the aggregation kernels.
// Sites may live on different devices of this process: every site has a device label, the buffers of a site are allocated on its
// device, its aggregations launched there, and a transfer is a copy from the source's device to the destination's. The two
// relations live on the HOME device (the one current at creation): atoms of sites elsewhere are sliced into a staging area at
// home and sent to their sites before the program starts, and the aggregates a function spec elsewhere ends with are brought
// home before recompose. Labels beyond the visible devices wrap around, which runs every one of these paths on fewer GPUs.
struct ExPlace {
    int label;            // device label of the buffer's site
    int64_t off;          // offset in that label's pool
    int64_t stage = -1;   // offset of its staging copy in the home pool (buffers that decompose fills or recompose reads, away from home)
};
struct ja_exchange_plan {
    ExBuild B;
    std::vector<ExPlace> place;               // per buffer
    std::map<int, char*> pool;                // per label
    std::map<int, int> phys;                  // label -> device ordinal
    std::map<int, int> site_label;
    int home = 0;                             // label of the home device
    int64_t table_off = 0;                    // box tables, in the home pool
    std::map<int, cudaStream_t> stream;       // per site
    std::vector<cudaEvent_t> ready;           // per buffer: written
    std::map<int, cudaEvent_t> done;          // per site: its last step issued
    cudaEvent_t start = nullptr;
    char* at(int b) const { return pool.at(place[b].label) + place[b].off; }
};

extern "C" void ja_exchange_plan_destroy(ja_exchange_plan_t* p) {
    if (!p) return;
    int cur = 0;
    cudaGetDevice(&cur);
    for (auto& kv : p->stream) cudaStreamDestroy(kv.second);
    for (cudaEvent_t e : p->ready)
        if (e) cudaEventDestroy(e);
    for (auto& kv : p->done) cudaEventDestroy(kv.second);
    if (p->start) cudaEventDestroy(p->start);
    for (auto& kv : p->pool)
        if (kv.second) {
            cudaSetDevice(p->phys[kv.first]);
            cudaFree(kv.second);
        }
    cudaSetDevice(cur);
    delete p;
}

extern "C" ja_status_t ja_exchange_plan_create_on(const ja_exprog_t* prog, const ja_relation_t* partials, const int32_t* copy_site,
                                                  const int32_t* consumer_specs, int32_t n_specs, ja_agg_t agg, ja_relation_t* dst,
                                                  const int32_t* site_device, int32_t n_site_device, int64_t* stats,
                                                  ja_exchange_plan_t** out) {
    if (!out) return ja_fail(JA_ERR_INVALID_ARG, "null argument");
    ja_exchange_plan* p = new ja_exchange_plan();
    ja_status_t st = build_exchange(prog, partials, copy_site, consumer_specs, n_specs, agg, dst, &p->B);
    if (st != JA_OK) {
        delete p;
        return st;
    }
    ExBuild& B = p->B;
    int home_dev = 0, n_dev = 1;
    cudaError_t e = cudaGetDevice(&home_dev);
    if (e == cudaSuccess) e = cudaGetDeviceCount(&n_dev);
    if (e != cudaSuccess || n_dev < 1) {
        delete p;
        return ja_fail(JA_ERR_CUDA, "exchange plan: no device");
    }
    // labels: the home device's own ordinal is its label; a site without an entry lives at home
    p->home = home_dev;
    p->phys[p->home] = home_dev;
    for (int s : prog->gpus) {
        int label = p->home;
        if (site_device && s < n_site_device) {
            if (site_device[s] < 0) {
                delete p;
                return ja_fail(JA_ERR_INVALID_ARG, "site %d: negative device label", s);
            }
            label = site_device[s];
        }
        p->site_label[s] = label;
        p->phys[label] = label % n_dev;
    }
    // place every buffer in its site's pool; staging at home for what decompose fills or recompose reads away from home
    std::map<int, int64_t> size;
    auto take = [&](int label, int64_t bytes) {
        const int64_t off = size[label];
        size[label] += (bytes + 255) / 256 * 256;
        return off;
    };
    p->place.resize(B.bufs.size());
    for (size_t b = 0; b < B.bufs.size(); ++b) {
        p->place[b].label = p->site_label.at(B.bufs[b].site);
        p->place[b].off = take(p->place[b].label, B.bufs[b].bytes);
    }
    for (int a = 0; a < B.n_in; ++a)
        if (p->place[a].label != p->home) p->place[a].stage = take(p->home, B.bufs[a].bytes);
    for (int b : B.out_box_buf)
        if (p->place[b].label != p->home && p->place[b].stage < 0) p->place[b].stage = take(p->home, B.bufs[b].bytes);
    p->table_off = take(p->home, B.table_bytes);
    // the boxes address the home pool: a buffer at home directly, one elsewhere through its staging copy
    for (int i = 0; i < B.n_in; ++i) B.boxes[i].dst_off = p->place[i].stage >= 0 ? p->place[i].stage : p->place[i].off;
    for (int i = 0; i < B.n_out; ++i) {
        const ExPlace& pl = p->place[B.out_box_buf[i]];
        B.boxes[B.n_in + i].src_off = pl.stage >= 0 ? pl.stage : pl.off;
    }
    B.scratch = 0;
    for (auto& kv : size) B.scratch += kv.second;
    for (auto& kv : size) {
        if (e != cudaSuccess) break;
        e = cudaSetDevice(p->phys[kv.first]);
        char* mem = nullptr;
        if (e == cudaSuccess) e = cudaMalloc((void**)&mem, (size_t)std::max<int64_t>(kv.second, 256));
        if (e == cudaSuccess) p->pool[kv.first] = mem;
    }
    if (e == cudaSuccess) e = cudaSetDevice(home_dev);
    if (e == cudaSuccess) e = cudaMemcpy(p->pool[p->home] + p->table_off, B.boxes.data(), (size_t)B.table_bytes, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->start, cudaEventDisableTiming);
    p->ready.assign(B.bufs.size(), nullptr);
    for (size_t i = 0; e == cudaSuccess && i < B.bufs.size(); ++i)
        if (B.bufs[i].producer_site >= 0) {
            e = cudaSetDevice(p->phys[p->site_label.at(B.bufs[i].producer_site)]);      // recorded on the producer's stream
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ready[i], cudaEventDisableTiming);
        }
    for (size_t i = 0; e == cudaSuccess && i < B.sites.size(); ++i) {
        e = cudaSetDevice(p->phys[p->site_label.at(B.sites[i])]);
        cudaStream_t s = nullptr;
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking);
        if (e == cudaSuccess) p->stream[B.sites[i]] = s;
        cudaEvent_t ev = nullptr;
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
        if (e == cudaSuccess) p->done[B.sites[i]] = ev;
    }
    cudaSetDevice(home_dev);
    if (e != cudaSuccess) {
        ja_exchange_plan_destroy(p);
        return ja_fail(e == cudaErrorMemoryAllocation ? JA_ERR_OOM : JA_ERR_CUDA, "exchange plan: %s", cudaGetErrorString(e));
    }
    fill_stats(B, stats);
    *out = p;
    return JA_OK;
}

extern "C" ja_status_t ja_exchange_plan_create(const ja_exprog_t* prog, const ja_relation_t* partials, const int32_t* copy_site,
                                               const int32_t* consumer_specs, int32_t n_specs, ja_agg_t agg, ja_relation_t* dst,
                                               int64_t* stats, ja_exchange_plan_t** out) {
    return ja_exchange_plan_create_on(prog, partials, copy_site, consumer_specs, n_specs, agg, dst, nullptr, 0, stats, out);
}

namespace {
// a device switch only when the device changes
cudaError_t set_device_if(int dev) {
    int cur = -1;
    cudaError_t e = cudaGetDevice(&cur);
    if (e != cudaSuccess) return e;
    return cur == dev ? cudaSuccess : cudaSetDevice(dev);
}
// Between two buffers of this process, on one device or two: under unified addressing the runtime finds the devices from the
// pointers, and the copy can be recorded by a stream capture (cudaMemcpyPeerAsync cannot: a capture that meets it is invalidated).
cudaError_t copy_between(void* dst, const void* src, size_t bytes, cudaStream_t st) {
    return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, st);
}
}  // namespace

extern "C" ja_status_t ja_exchange_plan_run(ja_exchange_plan_t* p, void* cuda_stream) {
    if (!p) return ja_fail(JA_ERR_INVALID_ARG, "null plan");
    const ExBuild& B = p->B;
    cudaStream_t user = (cudaStream_t)cuda_stream;
    const int home_dev = p->phys.at(p->home);
    int cur = 0;
    JA_CUDA(cudaGetDevice(&cur));
    if (cur != home_dev) return ja_fail(JA_ERR_INVALID_ARG, "the plan was created with device %d current, now it is %d", home_dev, cur);
    char* home = p->pool.at(p->home);
    const JaBoxCopy* d_boxes = (const JaBoxCopy*)(home + p->table_off);
    struct Restore {
        int dev;
        ~Restore() { set_device_if(dev); }
    } restore{cur};
    auto dev_of = [&](int b) { return p->phys.at(p->place[b].label); };
    ja_status_t rc = ja_launch_box_copies(B.src_base, home, d_boxes, B.n_in, B.max_in, B.vec_in, B.esize, user);
    if (rc != JA_OK) return rc;
    for (int a = 0; a < B.n_in; ++a)          // atoms of sites on other devices leave home
        if (p->place[a].stage >= 0)
            JA_CUDA(copy_between(p->at(a), home + p->place[a].stage, (size_t)B.bufs[a].bytes, user));
    if (!B.steps.empty()) {
        // fork: every site's stream starts after decompose
        JA_CUDA(cudaEventRecord(p->start, user));
        for (auto& kv : p->stream) JA_CUDA(cudaStreamWaitEvent(kv.second, p->start, 0));
        for (const ExStep& s : B.steps) {
            cudaStream_t st = p->stream.at(s.site);
            for (int b : s.parts)
                if (B.bufs[b].producer_site >= 0 && B.bufs[b].producer_site != s.site) JA_CUDA(cudaStreamWaitEvent(st, p->ready[b], 0));
            if (s.parts.size() == 1 && B.bufs[s.out].producer_site >= 0 && B.bufs[s.out].producer_site != s.site)
                JA_CUDA(cudaStreamWaitEvent(st, p->ready[s.out], 0));
            JA_CUDA(set_device_if(dev_of(s.out)));
            char* here = p->at(s.out);
            if (s.parts.size() >= 2) {
                const void* parts[JA_EXCHANGE_MAX_PARTS];
                for (size_t k = 0; k < s.parts.size(); ++k) parts[k] = p->at(s.parts[k]);
                if ((rc = ja_launch_exchange_combine(parts, (int)s.parts.size(), here, B.bufs[s.out].bytes, B.dtype, B.agg, st)) != JA_OK) return rc;
                JA_CUDA(cudaEventRecord(p->ready[s.out], st));
            }
            for (int d : s.dests) {
                JA_CUDA(copy_between(p->at(d), here, (size_t)B.bufs[s.out].bytes, st));
                JA_CUDA(cudaEventRecord(p->ready[d], st));
            }
        }
        // join
        JA_CUDA(set_device_if(home_dev));
        for (auto& kv : p->stream) {
            JA_CUDA(cudaEventRecord(p->done.at(kv.first), kv.second));
            JA_CUDA(cudaStreamWaitEvent(user, p->done.at(kv.first), 0));
        }
    }
    std::set<int> brought;
    for (int b : B.out_box_buf)              // what function specs on other devices ended with comes home
        if (p->place[b].stage >= 0 && brought.insert(b).second)
            JA_CUDA(copy_between(home + p->place[b].stage, p->at(b), (size_t)B.bufs[b].bytes, user));
    return ja_launch_box_copies(home, B.dst_base, d_boxes + B.n_in, B.n_out, B.max_out, B.vec_out, B.esize, user);
}
