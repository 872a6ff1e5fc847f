// Host-side lowering of an operator tree (paper Section 3.2: Sequence / Wait / Write /
// IfElse / DoWhile) to a byte-level deterministic transition table.
//
// Construction: every operator is lowered against a CONTINUATION state k (where control
// goes once the operator's language has been matched) and returns its ENTRY state.  A
// Sequence folds its parts from the right; a Write is a chain of one-symbol states ending in
// k; a Wait or Switch is one state whose deciding symbols lead to the entry of the chosen
// body lowered against k and whose stay symbols loop; a DoWhile first allocates its
// condition state c, lowers the body against c, and wires c's true symbols back to the
// body's entry and its false symbols to k.  An absent body contributes nothing (its entry
// is its continuation).  Because the deciding sets of one primitive are disjoint the result
// is deterministic without a subset construction.  States are then renumbered breadth-first
// from the start state and the 257 symbols are merged into classes with equal columns.
#include <algorithm>
#include <cstring>
#include <queue>
#include <unordered_map>
#include <utility>

#include "wg_internal.h"

namespace {

struct SymSet {
    uint32_t w[WG_SET_WORDS];
    bool has(int s) const { return (w[s >> 5] >> (s & 31)) & 1u; }
    bool empty() const {
        for (uint32_t x : w) if (x) return false;
        return true;
    }
    bool meets(const SymSet &o) const {
        for (int i = 0; i < WG_SET_WORDS; ++i) if (w[i] & o.w[i]) return true;
        return false;
    }
};

struct Edge {
    SymSet on;
    int32_t to;
};

struct Lowerer {
    const wg_op_node *nodes;
    int32_t n_nodes;
    const int32_t *children;
    const SymSet *sets;
    const uint8_t *data;
    std::vector<std::vector<Edge>> states;  // outgoing edges; symbols on no edge go to DEAD
    std::vector<int32_t> forced_tok, forced_next;  // per state; -1 = an ordinary state
    std::vector<wg_hole_site> holes;               // placeholder states of a template

    int32_t new_state() {
        states.emplace_back();
        forced_tok.push_back(-1);
        forced_next.push_back(0);
        return (int32_t)states.size() - 1;
    }

    static SymSet single(int sym) {
        SymSet s{};
        s.w[sym >> 5] = 1u << (sym & 31);
        return s;
    }

    // stay = (allow \ deny) \ (union of the deciding sets)
    SymSet stay_set(const wg_op_node &n) const {
        SymSet s = sets[n.set_off];
        const SymSet &deny = sets[n.set_off + 1];
        for (int i = 0; i < WG_SET_WORDS; ++i) s.w[i] &= ~deny.w[i];
        for (int d = 2; d < n.n_set; ++d)
            for (int i = 0; i < WG_SET_WORDS; ++i) s.w[i] &= ~sets[n.set_off + d].w[i];
        return s;
    }

    int32_t lower(int32_t node, int32_t k) {
        if (node < 0) return k;
        const wg_op_node &n = nodes[node];
        switch (n.kind) {
        case WG_OP_SEQUENCE: {
            int32_t next = k;
            for (int j = n.n_child - 1; j >= 0; --j) next = lower(children[n.child_off + j], next);
            return next;
        }
        case WG_OP_WRITE: {
            int32_t next = k;
            for (int j = n.data_len - 1; j >= 0; --j) {
                int32_t s = new_state();
                states[s].push_back({single(data[n.data_off + j]), next});
                next = s;
            }
            return next;
        }
        case WG_OP_WAIT:
        case WG_OP_SWITCH: {
            int32_t s = new_state();
            for (int c = 0; c < n.n_child; ++c) {
                int32_t target = lower(children[n.child_off + c], k);
                states[s].push_back({sets[n.set_off + 2 + c], target});
            }
            SymSet stay = stay_set(n);
            if (!stay.empty()) states[s].push_back({stay, s});
            return s;
        }
        case WG_OP_HOLE: {
            // A placeholder with no way out; instantiation replaces it by the entry of the
            // argument's automaton lowered against k.
            const int32_t s = new_state();
            holes.push_back({s, n.reserved, k});
            return s;
        }
        case WG_OP_WRITE_TOKENS: {
            // One state per forced token: no byte leaves it, only the token id itself.
            int32_t next = k;
            for (int j = n.data_len / 4 - 1; j >= 0; --j) {
                int32_t tok;
                memcpy(&tok, data + n.data_off + 4 * j, 4);
                const int32_t s = new_state();
                forced_tok[s] = tok;
                forced_next[s] = next;
                next = s;
            }
            return next;
        }
        case WG_OP_WAIT_UNTIL: {
            // One state per length of matched prefix of the string u (0 .. len-1), wired as
            // the string-matching automaton of u: from "k bytes matched", byte b leads to the
            // longest prefix of u that is a suffix of u[0..k) + b, found through the failure
            // links.  Reaching the full length enters the body.
            const uint8_t *u = data + n.data_off;
            const int len = n.data_len;
            std::vector<int> fail(len, 0);
            for (int i = 1, m = 0; i < len; ++i) {
                while (m > 0 && u[i] != u[m]) m = fail[m - 1];
                if (u[i] == u[m]) ++m;
                fail[i] = m;
            }
            std::vector<int32_t> st(len);
            for (int i = 0; i < len; ++i) st[i] = new_state();
            const int32_t done = lower(children[n.child_off], k);
            SymSet ok = sets[n.set_off];
            for (int i = 0; i < WG_SET_WORDS; ++i) ok.w[i] &= ~sets[n.set_off + 1].w[i];
            for (int i = 0; i < len; ++i) ok.w[u[i] >> 5] |= 1u << (u[i] & 31);
            for (int at = 0; at < len; ++at) {
                std::vector<SymSet> to(len + 1, SymSet{});
                for (int b = 0; b < 256; ++b) {
                    if (!ok.has(b)) continue;
                    int j = at;
                    while (j > 0 && u[j] != (uint8_t)b) j = fail[j - 1];
                    if (u[j] == (uint8_t)b) ++j;
                    to[j].w[b >> 5] |= 1u << (b & 31);
                }
                if (ok.has(WG_SYM_EOS)) to[0].w[WG_SYM_EOS >> 5] |= 1u << (WG_SYM_EOS & 31);
                for (int j = 0; j <= len; ++j)
                    if (!to[j].empty()) states[st[at]].push_back({to[j], j == len ? done : st[j]});
            }
            return st[0];
        }
        default: {  // WG_OP_DOWHILE
            int32_t c = new_state();
            int32_t entry = lower(children[n.child_off], c);
            states[c].push_back({sets[n.set_off + 2], entry});
            states[c].push_back({sets[n.set_off + 3], k});
            SymSet stay = stay_set(n);
            if (!stay.empty()) states[c].push_back({stay, c});
            return entry;
        }
        }
    }
};

int32_t validate(const wg_op_node *nodes, int32_t n_nodes, const int32_t *children,
                 int32_t n_children, const SymSet *sets, int32_t n_sets, const uint8_t *data,
                 int32_t n_data, int32_t root, bool allow_holes) {
    std::vector<uint8_t> used(n_nodes, 0);
    used[root] = 1;
    for (int32_t i = 0; i < n_nodes; ++i) {
        const wg_op_node &n = nodes[i];
        if (n.n_child < 0 || n.child_off < 0 || (int64_t)n.child_off + n.n_child > n_children)
            return WG_ERR_ARG;
        if (n.n_set < 0 || n.set_off < 0 || (int64_t)n.set_off + n.n_set > n_sets) return WG_ERR_ARG;
        if (n.data_len < 0 || n.data_off < 0 || (int64_t)n.data_off + n.data_len > n_data)
            return WG_ERR_ARG;
        bool shape_ok = false;
        switch (n.kind) {
        case WG_OP_SEQUENCE: shape_ok = n.n_set == 0; break;
        case WG_OP_WRITE: shape_ok = n.n_child == 0 && n.n_set == 0; break;
        case WG_OP_WAIT: shape_ok = n.n_child == 1 && n.n_set == 3; break;
        case WG_OP_SWITCH: shape_ok = n.n_set >= 3 && n.n_child == n.n_set - 2; break;
        case WG_OP_DOWHILE: shape_ok = n.n_child == 1 && n.n_set == 4; break;
        case WG_OP_WAIT_UNTIL: shape_ok = n.n_child == 1 && n.n_set == 2; break;
        case WG_OP_WRITE_TOKENS: shape_ok = n.n_child == 0 && n.n_set == 0 && n.data_len % 4 == 0; break;
        case WG_OP_HOLE:
            if (!allow_holes) return WG_ERR_GRAMMAR;  // holes exist in templates only
            shape_ok = n.n_child == 0 && n.n_set == 0 && n.data_len == 0 && n.reserved >= 0;
            break;
        default: break;
        }
        if (!shape_ok) return WG_ERR_ARG;
        for (int j = 0; j < n.n_child; ++j) {
            int32_t c = children[n.child_off + j];
            if (c == -1) {
                if (n.kind == WG_OP_SEQUENCE) return WG_ERR_ARG;
                continue;
            }
            if (c < 0 || c >= n_nodes) return WG_ERR_ARG;
            if (used[c]) return WG_ERR_GRAMMAR;  // a node reached twice: not a tree
            used[c] = 1;
        }
        if (n.kind == WG_OP_WRITE_TOKENS) {
            for (int j = 0; j < n.data_len / 4; ++j) {
                int32_t tok;
                memcpy(&tok, data + n.data_off + 4 * j, 4);
                if (tok < 0) return WG_ERR_GRAMMAR;
            }
        }
        if (n.kind == WG_OP_WAIT_UNTIL) {
            if (n.data_len < 1) return WG_ERR_GRAMMAR;
            for (int j = 0; j < n.data_len; ++j)
                if (sets[n.set_off + 1].has(data[n.data_off + j])) return WG_ERR_GRAMMAR;
        }
        if (n.kind == WG_OP_WAIT || n.kind == WG_OP_SWITCH || n.kind == WG_OP_DOWHILE) {
            const SymSet &deny = sets[n.set_off + 1];
            for (int a = 2; a < n.n_set; ++a) {
                const SymSet &sa = sets[n.set_off + a];
                if (sa.empty() || sa.meets(deny)) return WG_ERR_GRAMMAR;
                for (int b = a + 1; b < n.n_set; ++b)
                    if (sa.meets(sets[n.set_off + b])) return WG_ERR_GRAMMAR;
            }
        }
    }
    for (int32_t i = 0; i < n_nodes; ++i)
        if (!used[i]) return WG_ERR_GRAMMAR;  // a node that hangs nowhere
    return WG_OK;
}

// A multiplicative hash over 8-byte words in four independent lanes (the tables hashed here are
// megabytes; one dependent multiply chain per 8 bytes was a sixth of the lowering time), folded
// together at the end; the last bytes go through byte-wise FNV-1a.
static uint64_t fnv1a_bytes(uint64_t h, const void *p, size_t n) {
    const uint8_t *b = (const uint8_t *)p;
    const uint64_t P = 0x100000001B3ull;
    uint64_t lane[4] = {h, h ^ 0x9E3779B97F4A7C15ull, h ^ 0xC2B2AE3D27D4EB4Full, h ^ 0x165667B19E3779F9ull};
    size_t i = 0;
    for (; i + 32 <= n; i += 32) {
        uint64_t w[4];
        memcpy(w, b + i, 32);
        for (int k = 0; k < 4; ++k) {
            lane[k] = (lane[k] ^ w[k]) * P;
            lane[k] ^= lane[k] >> 29;
        }
    }
    h = lane[0];
    for (int k = 1; k < 4; ++k) h = ((h ^ lane[k]) * P) ^ (h >> 31);
    for (; i < n; ++i) h = (h ^ b[i]) * P;
    return h;
}

}  // namespace

uint64_t wg_grammar_content_hash(const wg_grammar &g) {
    uint64_t h = 0xCBF29CE484222325ull;
    if (!g.forced_tok.empty()) {
        h = fnv1a_bytes(h, g.forced_tok.data(), g.forced_tok.size() * sizeof(int32_t));
        h = fnv1a_bytes(h, g.forced_next.data(), g.forced_next.size() * sizeof(int32_t));
    }
    h = fnv1a_bytes(h, &g.n_states, 4);
    h = fnv1a_bytes(h, &g.n_classes, 4);
    h = fnv1a_bytes(h, &g.done, 4);
    h = fnv1a_bytes(h, &g.eos_class, 4);
    h = fnv1a_bytes(h, g.byte_class, 256);
    h = fnv1a_bytes(h, g.table.data(), g.table.size() * sizeof(int32_t));
    return h;
}

int32_t wg_lower_tree(const wg_op_node *nodes, int32_t n_nodes, const int32_t *children,
                      int32_t n_children, const uint32_t *sets_raw, int32_t n_sets,
                      const uint8_t *data, int32_t n_data, int32_t root, wg_grammar *out,
                      std::vector<wg_hole_site> *sites) {
    if (!nodes || n_nodes <= 0 || root < 0 || root >= n_nodes || n_children < 0 || n_sets < 0 ||
        n_data < 0 || (n_children > 0 && !children) || (n_sets > 0 && !sets_raw) ||
        (n_data > 0 && !data))
        return WG_ERR_ARG;
    const SymSet *sets = reinterpret_cast<const SymSet *>(sets_raw);
    int32_t rc = validate(nodes, n_nodes, children, n_children, sets, n_sets, data, n_data, root,
                          sites != nullptr);
    if (rc != WG_OK) return rc;

    bool mentions_eos = false;
    for (int32_t s = 0; s < n_sets; ++s) mentions_eos |= sets[s].has(WG_SYM_EOS);

    Lowerer lw{nodes, n_nodes, children, sets, data, {}, {}, {}, {}};
    const int32_t dead = lw.new_state();  // 0: no edges
    (void)dead;
    const int32_t done = lw.new_state();
    lw.states[done].push_back({Lowerer::single(WG_SYM_EOS), done});
    int32_t k = done;
    if (!mentions_eos) {  // the implicit trailing EOS
        k = lw.new_state();
        lw.states[k].push_back({Lowerer::single(WG_SYM_EOS), done});
    }
    const int32_t start = lw.lower(root, k);

    // breadth-first renumbering from the start state; DEAD stays 0
    const int32_t n_raw = (int32_t)lw.states.size();
    std::vector<int32_t> hole_next(n_raw, -1);
    for (const wg_hole_site &h : lw.holes) hole_next[h.state] = h.next;
    std::vector<int32_t> new_id(n_raw, -1);
    std::vector<int32_t> order;
    order.reserve(n_raw);
    new_id[0] = 0;
    order.push_back(0);
    std::queue<int32_t> q;
    new_id[start] = 1;
    order.push_back(start);
    q.push(start);
    while (!q.empty()) {
        int32_t s = q.front();
        q.pop();
        for (const Edge &e : lw.states[s]) {
            if (new_id[e.to] < 0) {
                new_id[e.to] = (int32_t)order.size();
                order.push_back(e.to);
                q.push(e.to);
            }
        }
        if (lw.forced_tok[s] >= 0 && new_id[lw.forced_next[s]] < 0) {
            new_id[lw.forced_next[s]] = (int32_t)order.size();
            order.push_back(lw.forced_next[s]);
            q.push(lw.forced_next[s]);
        }
        if (hole_next[s] >= 0 && new_id[hole_next[s]] < 0) {  // what follows a hole is reachable
            new_id[hole_next[s]] = (int32_t)order.size();
            order.push_back(hole_next[s]);
            q.push(hole_next[s]);
        }
    }
    if (new_id[done] < 0) {  // cannot happen for a valid tree, but keep DONE addressable
        new_id[done] = (int32_t)order.size();
        order.push_back(done);
    }
    const int32_t S = (int32_t)order.size();

    // Symbol classes: two symbols share a class when they belong to exactly the same edge
    // sets, which makes their columns equal in every state.  The refinement runs over the
    // DISTINCT sets only (a few hundred even for tables with 10^5 states, where most states
    // are one-byte steps of a literal).
    std::vector<int32_t> cls(WG_N_SYMBOLS, 0);
    int32_t n_cls = 1;
    std::vector<SymSet> distinct;    // the distinct edge sets
    std::vector<int32_t> edge_set;   // for every edge, in the order walked below: its set's index
    {
        struct SetHash {
            size_t operator()(const SymSet &x) const {
                uint64_t h = 0xCBF29CE484222325ull;
                for (uint32_t w : x.w) h = (h ^ w) * 0x100000001B3ull;
                return (size_t)h;
            }
        };
        struct SetEq {
            bool operator()(const SymSet &a, const SymSet &b) const {
                return memcmp(a.w, b.w, sizeof(a.w)) == 0;
            }
        };
        std::unordered_map<SymSet, int, SetHash, SetEq> seen;
        std::vector<int32_t> renum;
        std::vector<int32_t> class_size(1, WG_N_SYMBOLS);
        for (int32_t i = 0; i < S; ++i) {
            for (const Edge &e : lw.states[order[i]]) {
                const auto ins = seen.emplace(e.on, (int)distinct.size());
                edge_set.push_back(ins.first->second);
                if (!ins.second) continue;
                distinct.push_back(e.on);
                // a one-symbol set (a literal's byte, a branch of an enum: most sets) only takes
                // its symbol out of the class it shares with others
                int members = 0, only = -1;
                for (int wi = 0; wi < WG_SET_WORDS; ++wi)
                    if (e.on.w[wi]) { members += __builtin_popcount(e.on.w[wi]); only = wi * 32 + __builtin_ctz(e.on.w[wi]); }
                if (members == 1) {
                    if (class_size[cls[only]] > 1) {
                        --class_size[cls[only]];
                        cls[only] = n_cls++;
                        class_size.push_back(1);
                    }
                    continue;
                }
                renum.assign((size_t)n_cls * 2, -1);
                int32_t n_next = 0;
                for (int sym = 0; sym < WG_N_SYMBOLS; ++sym) {
                    const int32_t key = cls[sym] * 2 + (e.on.has(sym) ? 1 : 0);
                    if (renum[key] < 0) renum[key] = n_next++;
                    cls[sym] = renum[key];
                }
                n_cls = n_next;
                class_size.assign(n_cls, 0);
                for (int sym = 0; sym < WG_N_SYMBOLS; ++sym) ++class_size[cls[sym]];
            }
        }
    }
    // class ids in order of first appearance over the byte values, EOS last
    {
        std::vector<int32_t> remap(n_cls, -1);
        int32_t n = 0;
        for (int sym = 0; sym < WG_N_SYMBOLS; ++sym)
            if (remap[cls[sym]] < 0) remap[cls[sym]] = n++;
        for (int sym = 0; sym < WG_N_SYMBOLS; ++sym) cls[sym] = remap[cls[sym]];
    }

    out->n_states = S;
    out->n_classes = n_cls;
    out->start = 1;
    out->done = new_id[done];
    out->eos_class = cls[WG_SYM_EOS];
    for (int b = 0; b < 256; ++b) out->byte_class[b] = (uint8_t)cls[b];
    out->table.assign((size_t)S * n_cls, 0);
    std::vector<int32_t> rep(n_cls, -1);  // one representative symbol per class
    for (int sym = 0; sym < WG_N_SYMBOLS; ++sym)
        if (rep[cls[sym]] < 0) rep[cls[sym]] = sym;
    // Every edge set is a union of classes: list them once per distinct set, then a state's row
    // is filled edge by edge (a literal state writes one cell instead of testing every class).
    std::vector<std::vector<int32_t>> set_classes(distinct.size());
    for (size_t d = 0; d < distinct.size(); ++d)
        for (int32_t c = 0; c < n_cls; ++c)
            if (distinct[d].has(rep[c])) set_classes[d].push_back(c);
    size_t edge_no = 0;
    for (int32_t i = 0; i < S; ++i) {
        const std::vector<Edge> &edges = lw.states[order[i]];
        int32_t *row = &out->table[(size_t)i * n_cls];
        // last edge first, so that where two edges of a state overlap the first one wins
        for (size_t k = edges.size(); k-- > 0;) {
            const int32_t to = new_id[edges[k].to];
            for (int32_t c : set_classes[edge_set[edge_no + k]]) row[c] = to;
        }
        edge_no += edges.size();
    }
    out->forced_tok.clear();
    out->forced_next.clear();
    bool any_forced = false;
    for (int32_t i = 0; i < S; ++i) any_forced |= lw.forced_tok[order[i]] >= 0;
    if (any_forced) {
        out->forced_tok.assign(S, -1);
        out->forced_next.assign(S, 0);
        for (int32_t i = 0; i < S; ++i) {
            if (lw.forced_tok[order[i]] < 0) continue;
            out->forced_tok[i] = lw.forced_tok[order[i]];
            out->forced_next[i] = new_id[lw.forced_next[order[i]]];
        }
    }
    out->tail = (!mentions_eos && new_id[k] >= 0) ? new_id[k] : -1;
    if (sites) {
        sites->clear();
        for (const wg_hole_site &h : lw.holes)
            if (new_id[h.state] >= 0)  // a hole that no path reaches needs no filling
                sites->push_back({new_id[h.state], h.arg, new_id[h.next]});
    }
    out->hash = wg_grammar_content_hash(*out);
    return WG_OK;
}

// Moore's partition refinement: start from {DEAD}, {DONE}, the forced-token states grouped by
// token id, and everything else; split blocks by the blocks their transitions lead to until
// nothing splits any more.  States of one final block accept the same continuations, so they
// get one state (and one cached mask) in the output.
int32_t wg_minimize_grammar(const wg_grammar &in, wg_grammar *out) {
    const int32_t S = in.n_states, C = in.n_classes;
    const bool forced = !in.forced_tok.empty();
    std::vector<int32_t> block(S, 0);
    int32_t n_blocks = 0;
    {
        std::unordered_map<int64_t, int32_t> first;
        for (int32_t s = 0; s < S; ++s) {
            int64_t key = s == 0 ? -1 : (s == in.done ? -2 : -3);
            if (s != 0 && forced && in.forced_tok[s] >= 0) key = in.forced_tok[s];
            auto it = first.find(key);
            if (it == first.end()) it = first.emplace(key, n_blocks++).first;
            block[s] = it->second;
        }
    }
    const int width = C + 2;
    std::vector<int32_t> sig((size_t)S * width);
    std::vector<int32_t> order(S), next_block(S);
    std::vector<std::pair<uint64_t, int32_t>> keyed(S);
    for (;;) {
        for (int32_t s = 0; s < S; ++s) {
            int32_t *row = &sig[(size_t)s * width];
            row[0] = block[s];
            for (int32_t c = 0; c < C; ++c) row[1 + c] = block[in.table[(size_t)s * C + c]];
            row[1 + C] = (forced && in.forced_tok[s] >= 0) ? block[in.forced_next[s]] : -1;
        }
        // states with equal signatures next to each other: sort by a hash of the row (sorting
        // the wide rows themselves took most of the time), then by the rows inside the rare runs
        // where different rows share a hash
        auto row_less = [&](int32_t a, int32_t b) {
            const int cmp = memcmp(&sig[(size_t)a * width], &sig[(size_t)b * width], sizeof(int32_t) * width);
            return cmp != 0 ? cmp < 0 : a < b;
        };
        for (int32_t s = 0; s < S; ++s) {
            uint64_t h = 0xCBF29CE484222325ull;
            const int32_t *row = &sig[(size_t)s * width];
            for (int i = 0; i < width; ++i) { h = (h ^ (uint32_t)row[i]) * 0x100000001B3ull; h ^= h >> 32; }
            keyed[s] = {h, s};
        }
        std::sort(keyed.begin(), keyed.end());
        for (int32_t s = 0; s < S; ++s) order[s] = keyed[s].second;
        for (int32_t i = 0; i < S;) {
            int32_t j = i + 1;
            bool mixed = false;
            while (j < S && keyed[j].first == keyed[i].first) {
                mixed |= memcmp(&sig[(size_t)order[j] * width], &sig[(size_t)order[i] * width],
                                sizeof(int32_t) * width) != 0;
                ++j;
            }
            if (mixed) std::sort(order.begin() + i, order.begin() + j, row_less);
            i = j;
        }
        int32_t n_next = 0;
        for (int32_t i = 0; i < S; ++i) {
            if (i > 0 && memcmp(&sig[(size_t)order[i] * width], &sig[(size_t)order[i - 1] * width],
                                sizeof(int32_t) * width) != 0)
                ++n_next;
            next_block[order[i]] = n_next;
        }
        ++n_next;
        block.swap(next_block);
        if (n_next == n_blocks) break;  // refinement only splits: an equal count is a fixpoint
        n_blocks = n_next;
    }
    // new ids in order of first appearance (the input is numbered breadth-first from the start
    // state, so locality survives); DEAD stays 0
    std::vector<int32_t> new_id(n_blocks, -1), rep;
    rep.reserve(n_blocks);
    for (int32_t s = 0; s < S; ++s)
        if (new_id[block[s]] < 0) { new_id[block[s]] = (int32_t)rep.size(); rep.push_back(s); }
    const int32_t M = (int32_t)rep.size();
    out->n_states = M;
    out->n_classes = C;
    out->start = new_id[block[in.start]];
    out->done = new_id[block[in.done]];
    out->tail = in.tail >= 0 ? new_id[block[in.tail]] : -1;
    out->eos_class = in.eos_class;
    memcpy(out->byte_class, in.byte_class, sizeof(in.byte_class));
    out->table.assign((size_t)M * C, 0);
    for (int32_t m = 0; m < M; ++m)
        for (int32_t c = 0; c < C; ++c)
            out->table[(size_t)m * C + c] = new_id[block[in.table[(size_t)rep[m] * C + c]]];
    out->forced_tok.clear();
    out->forced_next.clear();
    if (forced) {
        out->forced_tok.assign(M, -1);
        out->forced_next.assign(M, 0);
        for (int32_t m = 0; m < M; ++m)
            if (in.forced_tok[rep[m]] >= 0) {
                out->forced_tok[m] = in.forced_tok[rep[m]];
                out->forced_next[m] = new_id[block[in.forced_next[rep[m]]]];
            }
    }
    out->hash = wg_grammar_content_hash(*out);
    return WG_OK;
}
