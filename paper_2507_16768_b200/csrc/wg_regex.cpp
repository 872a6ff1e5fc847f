// Regular expression -> operator tree (paper Section 3.2, the paragraph on translating regular
// expressions into Wait / Write compositions; the syntax-prior variant evaluated in Section 4.1).
//
// Character classes and single characters become Wait operators, literal runs become Write,
// repetition and branching become DoWhile / IfElse(Switch) / Sequence.  Because the operators
// decide on ONE symbol and consume it, the translation exists only for patterns that are
// deterministic with one symbol of look-ahead: wherever a choice is made (leave a repetition
// or stay in it, which alternative to take) the candidate first symbols must not overlap.
// Such a pattern matches the same strings under greedy and non-greedy reading (paper
// Section 6).  Patterns outside this class are refused with WG_ERR_GRAMMAR and a message.
//
// Shape of the output for "X+ (G)* tail", which is the shape of the paper's worked example:
//   Wait(allow = X, wait = X)                       one X
//   Switch(allow = X | first(G) | first(tail),      further X stay here
//          first(tail) -> nothing,
//          first(G)    -> DoWhile(body = rest of G, cond(true = first(G), false = first(tail))))
//   rest of tail
#include <cstdio>
#include <cstring>
#include <memory>
#include <string>
#include <vector>

#include "wg_internal.h"

namespace {

struct Set {
    uint32_t w[WG_SET_WORDS] = {};
    void add(int s) { w[s >> 5] |= 1u << (s & 31); }
    bool has(int s) const { return (w[s >> 5] >> (s & 31)) & 1u; }
    bool empty() const { for (uint32_t x : w) if (x) return false; return true; }
    bool meets(const Set &o) const { for (int i = 0; i < WG_SET_WORDS; ++i) if (w[i] & o.w[i]) return true; return false; }
    bool subset_of(const Set &o) const { for (int i = 0; i < WG_SET_WORDS; ++i) if (w[i] & ~o.w[i]) return false; return true; }
    Set operator|(const Set &o) const { Set r; for (int i = 0; i < WG_SET_WORDS; ++i) r.w[i] = w[i] | o.w[i]; return r; }
    bool operator==(const Set &o) const { return memcmp(w, o.w, sizeof(w)) == 0; }
    int count() const { int n = 0; for (uint32_t x : w) n += __builtin_popcount(x); return n; }
    int lowest() const { for (int s = 0; s < WG_N_SYMBOLS; ++s) if (has(s)) return s; return -1; }
    void complement_bytes() { for (int i = 0; i < 8; ++i) w[i] = ~w[i]; }
};

// ---- syntax tree ------------------------------------------------------------------------
enum Kind { R_SET, R_CAT, R_ALT, R_STAR, R_PLUS, R_OPT };
struct Re {
    Kind kind;
    Set set;                // R_SET: the symbols, one of which is consumed
    std::vector<int> kids;  // indices into the arena
};

struct Fail { std::string msg; };

struct Parser {
    const unsigned char *p;
    int n, i = 0;
    std::vector<Re> &arena;
    int depth = 0;

    int make(Kind k) { arena.push_back(Re{k, Set{}, {}}); return (int)arena.size() - 1; }
    [[noreturn]] void fail(const std::string &m) { throw Fail{m + " at offset " + std::to_string(i)}; }
    bool more() const { return i < n; }

    static void add_range(Set &s, int lo, int hi) { for (int c = lo; c <= hi; ++c) s.add(c); }
    static Set digits() { Set s; add_range(s, '0', '9'); return s; }
    static Set word() { Set s = digits(); add_range(s, 'a', 'z'); add_range(s, 'A', 'Z'); s.add('_'); return s; }
    static Set space() { Set s; for (int c : {' ', '\t', '\n', '\r', '\f', '\v'}) s.add(c); return s; }

    int hex_digit() {
        if (!more()) fail("unfinished \\x escape");
        int c = p[i++];
        if (c >= '0' && c <= '9') return c - '0';
        if (c >= 'a' && c <= 'f') return c - 'a' + 10;
        if (c >= 'A' && c <= 'F') return c - 'A' + 10;
        fail("bad hex digit");
    }

    // after a backslash: a class (returns true, fills s) or a single byte (c)
    bool escape(Set &s, int &c) {
        if (!more()) fail("pattern ends with a backslash");
        int e = p[i++];
        switch (e) {
        case 'd': s = digits(); return true;
        case 'w': s = word(); return true;
        case 's': s = space(); return true;
        case 'D': s = digits(); s.complement_bytes(); return true;
        case 'W': s = word(); s.complement_bytes(); return true;
        case 'S': s = space(); s.complement_bytes(); return true;
        case 'n': c = '\n'; return false;
        case 't': c = '\t'; return false;
        case 'r': c = '\r'; return false;
        case 'f': c = '\f'; return false;
        case 'v': c = '\v'; return false;
        case '0': c = 0; return false;
        case 'x': { int h = hex_digit(); c = h * 16 + hex_digit(); return false; }
        default:
            if ((e >= 'a' && e <= 'z') || (e >= 'A' && e <= 'Z') || (e >= '1' && e <= '9'))
                fail(std::string("unsupported escape \\") + (char)e);
            c = e;
            return false;
        }
    }

    int parse_class() {  // after '['
        Set s;
        bool negate = false;
        if (more() && p[i] == '^') { negate = true; ++i; }
        bool first = true;
        for (;;) {
            if (!more()) fail("unterminated [ ]");
            int c = p[i++];
            if (c == ']' && !first) break;
            first = false;
            Set cls;
            bool is_class = false;
            if (c == '\\') is_class = escape(cls, c);
            if (is_class) { s = s | cls; continue; }
            if (i + 1 < n && p[i] == '-' && p[i + 1] != ']') {
                ++i;
                int hi = p[i++];
                if (hi == '\\') { Set dummy; if (escape(dummy, hi)) fail("class escape as range end"); }
                if (hi < c) fail("reversed range");
                add_range(s, c, hi);
            } else {
                s.add(c);
            }
        }
        if (negate) s.complement_bytes();
        if (s.empty()) fail("empty character class");
        int id = make(R_SET);
        arena[id].set = s;
        return id;
    }

    int parse_atom() {
        int c = p[i++];
        if (c == '(') {
            if (++depth > 64) fail("groups nested too deeply");
            if (i + 1 < n && p[i] == '?' && p[i + 1] == ':') i += 2;
            else if (more() && p[i] == '?') fail("unsupported group syntax (?...)");
            int g = parse_alt();
            if (!more() || p[i] != ')') fail("missing )");
            ++i;
            --depth;
            return g;
        }
        if (c == '[') return parse_class();
        int id = make(R_SET);
        if (c == '.') {
            arena[id].set.complement_bytes();  // all 256 bytes ...
            arena[id].set.w[0] &= ~(1u << '\n');  // ... except newline
            return id;
        }
        if (c == '\\') {
            Set s;
            if (escape(s, c)) { arena[id].set = s; return id; }
        } else if (c == '*' || c == '+' || c == '?' || c == '{' || c == '}' || c == ')' || c == ']' ||
                   c == '|' || c == '^' || c == '$') {
            --i;
            fail(std::string("unexpected '") + (char)c + "'");
        }
        arena[id].set.add(c);
        return id;
    }

    int copy(int node) {  // deep copy for counted repetition
        Re r = arena[node];
        for (int &k : r.kids) k = copy(k);
        arena.push_back(r);
        return (int)arena.size() - 1;
    }

    int unary(Kind k, int child) { int id = make(k); arena[id].kids = {child}; return id; }

    int parse_repeat() {
        int atom = parse_atom();
        while (more()) {
            int c = p[i];
            if (c == '*') { ++i; atom = unary(R_STAR, atom); }
            else if (c == '+') { ++i; atom = unary(R_PLUS, atom); }
            else if (c == '?') { ++i; atom = unary(R_OPT, atom); }
            else if (c == '{') {
                ++i;
                auto number = [&]() { int v = -1; while (more() && p[i] >= '0' && p[i] <= '9') { v = (v < 0 ? 0 : v) * 10 + (p[i++] - '0'); if (v > 1000) fail("repeat count too large"); } return v; };
                int lo = number(), hi = lo;
                if (lo < 0) fail("bad {m,n}");
                if (more() && p[i] == ',') { ++i; hi = number(); }  // hi < 0: unbounded
                if (!more() || p[i] != '}') fail("bad {m,n}");
                ++i;
                if (hi >= 0 && (hi < lo || hi > 64)) fail("bad or too large {m,n}");
                // X{m,n} = X^m followed by n-m nested optionals (X(X(...)?)?)?; X{m,} = X^m X*
                int cat = make(R_CAT);
                std::vector<int> kids;
                for (int k = 0; k < lo; ++k) kids.push_back(copy(atom));
                if (hi < 0) {
                    kids.push_back(unary(R_STAR, copy(atom)));
                } else if (hi > lo) {
                    int tail = -1;
                    for (int k = 0; k < hi - lo; ++k) {
                        int c2 = make(R_CAT);
                        std::vector<int> inner = {copy(atom)};
                        if (tail >= 0) inner.push_back(tail);
                        arena[c2].kids = inner;
                        tail = unary(R_OPT, c2);
                    }
                    kids.push_back(tail);
                }
                arena[cat].kids = kids;
                atom = cat;
            } else break;
            if (more() && p[i] == '?') ++i;  // lazy marker: same language, ignored
        }
        return atom;
    }

    int parse_cat() {
        int cat = make(R_CAT);
        std::vector<int> kids;
        while (more() && p[i] != '|' && p[i] != ')') {
            if (p[i] == '^' && i == 0) { ++i; continue; }         // anchors at the ends are implied
            if (p[i] == '$' && i == n - 1) { ++i; continue; }
            kids.push_back(parse_repeat());
        }
        arena[cat].kids = kids;
        return cat;
    }

    int parse_alt() {
        int first = parse_cat();
        if (!more() || p[i] != '|') return first;
        int alt = make(R_ALT);
        std::vector<int> kids = {first};
        while (more() && p[i] == '|') { ++i; kids.push_back(parse_cat()); }
        arena[alt].kids = kids;
        return alt;
    }
};

// ---- operator IR ------------------------------------------------------------------------
struct Op;
using Chain = std::vector<std::unique_ptr<Op>>;
struct Op {
    int kind;                  // WG_OP_*
    std::string literal;       // WRITE
    Set allow;                 // WAIT / SWITCH / DOWHILE
    std::vector<Set> cases;    // WAIT: [wait]; SWITCH: k sets; DOWHILE: [true, false]
    std::vector<Chain> bodies; // SWITCH: k chains (empty = absent); DOWHILE: [body]
};

struct Gen {
    std::vector<Re> &arena;
    size_t budget = 200000;  // operators; patterns that duplicate their tails too often stop here

    [[noreturn]] void fail(const std::string &m) { throw Fail{m}; }

    void flatten(int node, std::vector<int> &out) const {
        if (arena[node].kind == R_CAT) for (int k : arena[node].kids) flatten(k, out);
        else out.push_back(node);
    }
    std::vector<int> items_of(int node) const { std::vector<int> v; flatten(node, v); return v; }

    // An alternation of single-symbol sets is one set.
    bool as_set(int node, Set &s) const {
        const Re &r = arena[node];
        if (r.kind == R_SET) { s = r.set; return true; }
        if (r.kind == R_CAT && r.kids.size() == 1) return as_set(r.kids[0], s);
        if (r.kind == R_ALT) {
            Set u;
            for (int k : r.kids) { Set t; if (!as_set(k, t)) return false; u = u | t; }
            s = u;
            return true;
        }
        return false;
    }

    bool nullable(int node) const {
        const Re &r = arena[node];
        switch (r.kind) {
        case R_SET: return false;
        case R_STAR: case R_OPT: return true;
        case R_PLUS: return nullable(r.kids[0]);
        case R_CAT: for (int k : r.kids) if (!nullable(k)) return false; return true;
        default: for (int k : r.kids) if (nullable(k)) return true; return false;
        }
    }

    Set first_of(const std::vector<int> &items, size_t from = 0) const {
        Set f;
        for (size_t j = from; j < items.size(); ++j) {
            f = f | first_node(items[j]);
            if (!nullable(items[j])) break;
        }
        return f;
    }
    Set first_node(int node) const {
        const Re &r = arena[node];
        switch (r.kind) {
        case R_SET: return r.set;
        case R_CAT: return first_of(r.kids);
        case R_ALT: { Set f; for (int k : r.kids) f = f | first_node(k); return f; }
        default: return first_node(r.kids[0]);
        }
    }

    std::unique_ptr<Op> new_op(int kind) {
        if (budget-- == 0) fail("pattern expands to too many operators (optional parts duplicate what follows them)");
        auto op = std::make_unique<Op>();
        op->kind = kind;
        return op;
    }

    static void append(Chain &dst, Chain &&src) { for (auto &o : src) dst.push_back(std::move(o)); }

    void need_disjoint(const Set &a, const Set &b, const char *what) {
        if (a.meets(b)) fail(std::string("not decidable on one symbol: ") + what);
    }

    // One symbol of `take` has just been consumed from the front of items[from]; what is left
    // of that item is prepended to the items after it.  Only for items that start with a
    // plain set or with a literal run.
    // Emits the chain for `pending* items[from..]`; the symbols in `pending` may still arrive
    // (they belong to a class repetition that was entered earlier) and keep the next
    // decision where it is.  Returns the class repetition left open at the end, if any.
    Set gen(const std::vector<int> &items, size_t from, Set pending, Chain &out) {
        while (from < items.size()) {
            const int node = items[from];
            const Kind kind = arena[node].kind;
            const int kid0 = arena[node].kids.empty() ? -1 : arena[node].kids[0];
            Set s;
            if (kind == R_CAT) {
                std::vector<int> flat(items.begin(), items.begin() + from);
                flatten(node, flat);
                flat.insert(flat.end(), items.begin() + from + 1, items.end());
                return gen(flat, from, pending, out);
            }
            if (as_set(node, s)) {  // one symbol out of s; literal runs become one Write
                need_disjoint(pending, s, "a repeated class runs into the symbol that follows it");
                if (s.count() == 1 && s.lowest() < 256) {
                    std::string lit(1, (char)s.lowest());
                    size_t j = from + 1;
                    Set t;
                    while (j < items.size() && as_set(items[j], t) && t.count() == 1 && t.lowest() < 256) {
                        lit.push_back((char)t.lowest());
                        ++j;
                    }
                    if (!pending.empty()) {  // leave the repetition on the literal's first byte
                        auto w = new_op(WG_OP_WAIT);
                        w->allow = pending | s;
                        w->cases = {s};
                        out.push_back(std::move(w));
                        lit.erase(0, 1);
                    }
                    if (!lit.empty()) {
                        auto wr = new_op(WG_OP_WRITE);
                        wr->literal = lit;
                        out.push_back(std::move(wr));
                    }
                    from = j;
                } else {
                    auto w = new_op(WG_OP_WAIT);
                    w->allow = pending | s;
                    w->cases = {s};
                    out.push_back(std::move(w));
                    ++from;
                }
                pending = Set{};
                continue;
            }
            Set inner;
            const bool rep_of_set = (kind == R_PLUS || kind == R_STAR) && as_set(kid0, inner);
            if (rep_of_set && kind == R_PLUS) {  // C+ = one C, then more C may arrive
                need_disjoint(pending, inner, "two adjacent repetitions share symbols");
                auto w = new_op(WG_OP_WAIT);
                w->allow = pending | inner;
                w->cases = {inner};
                out.push_back(std::move(w));
                pending = inner;
                ++from;
                continue;
            }
            if (rep_of_set && pending.subset_of(inner)) {  // C*: nothing to consume yet
                pending = inner;
                ++from;
                continue;
            }
            if (kind == R_PLUS) {  // (G)+ = G (G)*
                std::vector<int> next(items.begin(), items.begin() + from);
                flatten(kid0, next);
                const int star = (int)arena.size();
                arena.push_back(Re{R_STAR, Set{}, {kid0}});
                next.push_back(star);
                next.insert(next.end(), items.begin() + from + 1, items.end());
                return gen(next, from, pending, out);
            }
            if (kind == R_STAR) return gen_star(items, from, pending, out);
            return gen_choice(items, from, pending, out);  // R_OPT, R_ALT
        }
        return pending;
    }

    // items[from] = (G)*.  Decide between one more G and leaving, on one symbol:
    //   Switch(leave -> nothing, first(G) -> DoWhile(rest of G, cond(true = first(G), false = leave)))
    // then the rest of the tail, whose first symbol the decision has consumed.
    Set gen_star(const std::vector<int> &items, size_t from, Set pending, Chain &out) {
        const int group = arena[items[from]].kids[0];
        std::vector<int> g = items_of(group);
        if (g.empty() || nullable(group)) fail("a repeated group must consume at least one symbol");
        if (from + 1 >= items.size()) fail("internal: repetition without a follower");
        const Set first_g = first_of(g);
        const Set leave = first_of(items, from + 1);
        need_disjoint(first_g, leave, "a repeated group and what follows it start with the same symbol");
        need_disjoint(pending, first_g, "a repeated class runs into the group that follows it");
        need_disjoint(pending, leave, "a repeated class runs into the symbol that follows it");
        // the body: G with its first symbol consumed; G must begin with a set or a literal
        Set g0;
        if (!as_set(g[0], g0) && !(arena[g[0]].kind == R_PLUS && as_set(arena[g[0]].kids[0], g0)))
            fail("a repeated group must begin with a character, a class or a repeated class");
        Chain body;
        Set body_pending;
        {
            std::vector<int> rest(g.begin() + 1, g.end());
            Set p0;
            if (arena[g[0]].kind == R_PLUS) p0 = g0;  // C+ ...: one C consumed, more may follow
            body_pending = gen(rest, 0, p0, body);
        }
        need_disjoint(body_pending, first_g, "a repeated group ends in a class that its own start overlaps");
        need_disjoint(body_pending, leave, "a repeated group ends in a class that the follower overlaps");
        auto loop = new_op(WG_OP_DOWHILE);
        loop->allow = body_pending | first_g | leave;
        loop->cases = {first_g, leave};
        loop->bodies.resize(1);
        loop->bodies[0] = std::move(body);
        auto sw = new_op(WG_OP_SWITCH);
        sw->allow = pending | first_g | leave;
        sw->cases = {leave, first_g};
        sw->bodies.resize(2);
        sw->bodies[1].push_back(std::move(loop));
        out.push_back(std::move(sw));
        return gen_after_first(items, from + 1, out);
    }

    // The first symbol of items[from..] has been consumed by a decision that could not tell
    // which symbol it was: legal only if what remains does not depend on it.
    Set gen_after_first(const std::vector<int> &items, size_t from, Chain &out) {
        const int node = items[from];
        const Re r = arena[node];
        Set s;
        if (as_set(node, s)) return gen(items, from + 1, Set{}, out);
        if (r.kind == R_PLUS && as_set(r.kids[0], s)) {  // C+ with one C consumed: C* remains
            return gen(items, from + 1, s, out);
        }
        if (r.kind == R_STAR && as_set(r.kids[0], s)) {
            // the consumed symbol was either a C (stay in C*) or the follower's first symbol
            fail("a repetition is followed by another optional repetition; add a separator");
        }
        if (r.kind == R_CAT) {
            std::vector<int> flat(items.begin(), items.begin() + from);
            flatten(node, flat);
            flat.insert(flat.end(), items.begin() + from + 1, items.end());
            return gen_after_first(flat, from, out);
        }
        fail("a repetition must be followed by a character, a class or a repeated class");
    }

    // items[from] is an alternation or an optional part: one Switch whose cases are the first
    // symbols of the alternatives (and, for an optional part, of what follows it).
    Set gen_choice(const std::vector<int> &items, size_t from, Set pending, Chain &out) {
        const Re r = arena[items[from]];
        struct Branch { std::vector<int> items; size_t own; };  // own = items that belong to the branch
        std::vector<Branch> branches;
        const std::vector<int> tail(items.begin() + from + 1, items.end());
        bool optional = r.kind == R_OPT;
        std::vector<int> alts;
        if (r.kind == R_OPT) {
            const Re inner = arena[r.kids[0]];
            if (inner.kind == R_ALT) alts = inner.kids; else alts = {r.kids[0]};
        } else {
            alts = r.kids;
        }
        for (int a : alts) {
            std::vector<int> b = items_of(a);
            if (b.empty() || nullable(a)) { optional = true; if (b.empty()) continue; }
            branches.push_back(Branch{b, b.size()});
        }
        if (optional && tail.empty()) fail("internal: optional part without a follower");
        // case sets
        std::vector<Set> firsts;
        Set all = pending;
        for (const Branch &b : branches) {
            Set f = first_of(b.items);
            need_disjoint(all, f, "two alternatives (or a class before them) start with the same symbol");
            all = all | f;
            firsts.push_back(f);
        }
        Set leave;
        if (optional) {
            leave = first_of(tail);
            need_disjoint(all, leave, "an optional part and what follows it start with the same symbol");
        }
        // First try: the branches alone, sharing the tail after the Switch.  That is right only
        // if no branch ends inside a class repetition and nothing is optional.
        auto sw = new_op(WG_OP_SWITCH);
        sw->allow = all | leave;
        bool share_tail = !optional;
        std::vector<Chain> bodies(branches.size());
        if (share_tail) {
            for (size_t k = 0; k < branches.size() && share_tail; ++k) {
                Set p = gen_branch(branches[k].items, bodies[k]);
                if (!p.empty()) share_tail = false;
            }
        }
        Set end_pending;
        if (!share_tail) {  // every branch carries its own copy of the tail
            bool first_branch = true;
            for (size_t k = 0; k < branches.size(); ++k) {
                bodies[k].clear();
                std::vector<int> full = branches[k].items;
                full.insert(full.end(), tail.begin(), tail.end());
                Set p = gen_branch(full, bodies[k]);
                if (!first_branch && !(p == end_pending)) fail("alternatives end in different open repetitions");
                end_pending = p;
                first_branch = false;
            }
        }
        for (size_t k = 0; k < branches.size(); ++k) {
            sw->cases.push_back(firsts[k]);
            sw->bodies.push_back(std::move(bodies[k]));
        }
        if (optional) {  // skipping the optional part: the decision has eaten the tail's first symbol
            Chain skip;
            Set p = gen_after_first(tail, 0, skip);
            if (!branches.empty() && !(p == end_pending)) fail("alternatives end in different open repetitions");
            end_pending = p;
            sw->cases.push_back(leave);
            sw->bodies.push_back(std::move(skip));
        }
        out.push_back(std::move(sw));
        if (share_tail) return gen(items, from + 1, Set{}, out);
        return end_pending;
    }

    // A branch whose first symbol (any of its first set) has been consumed by the Switch.
    Set gen_branch(const std::vector<int> &b, Chain &out) {
        Set s;
        const Re r0 = arena[b[0]];
        if (as_set(b[0], s)) return gen(b, 1, Set{}, out);
        if (r0.kind == R_PLUS && as_set(r0.kids[0], s)) return gen(b, 1, s, out);
        if (r0.kind == R_CAT) {
            std::vector<int> flat;
            flatten(b[0], flat);
            flat.insert(flat.end(), b.begin() + 1, b.end());
            return gen_branch(flat, out);
        }
        fail("an alternative must begin with a character, a class or a repeated class");
    }
};

// ---- flat arrays -------------------------------------------------------------------------
struct Flat {
    std::vector<wg_op_node> nodes;
    std::vector<int32_t> children;
    std::vector<uint32_t> sets;
    std::vector<uint8_t> data;

    int32_t add_sets(const std::vector<Set> &ss) {
        const int32_t off = (int32_t)(sets.size() / WG_SET_WORDS);
        for (const Set &s : ss) sets.insert(sets.end(), s.w, s.w + WG_SET_WORDS);
        return off;
    }

    int32_t emit_chain(const Chain &c) {
        if (c.empty()) return -1;
        if (c.size() == 1) return emit(*c[0]);
        const int32_t id = (int32_t)nodes.size();
        nodes.push_back(wg_op_node{WG_OP_SEQUENCE, (int32_t)c.size(), 0, 0, 0, 0, 0, 0});
        std::vector<int32_t> kids;
        for (const auto &o : c) kids.push_back(emit(*o));
        nodes[id].child_off = (int32_t)children.size();
        children.insert(children.end(), kids.begin(), kids.end());
        return id;
    }

    int32_t emit(const Op &o) {
        const int32_t id = (int32_t)nodes.size();
        nodes.push_back(wg_op_node{o.kind, 0, 0, 0, 0, 0, 0, 0});
        if (o.kind == WG_OP_WRITE) {
            nodes[id].data_off = (int32_t)data.size();
            nodes[id].data_len = (int32_t)o.literal.size();
            data.insert(data.end(), o.literal.begin(), o.literal.end());
            return id;
        }
        std::vector<Set> ss = {o.allow, Set{}};
        ss.insert(ss.end(), o.cases.begin(), o.cases.end());
        const int32_t set_off = add_sets(ss);
        std::vector<int32_t> kids;
        if (o.kind == WG_OP_WAIT) kids.push_back(-1);
        for (const Chain &b : o.bodies) kids.push_back(emit_chain(b));
        nodes[id].n_set = (int32_t)ss.size();
        nodes[id].set_off = set_off;
        nodes[id].n_child = (int32_t)kids.size();
        nodes[id].child_off = (int32_t)children.size();
        children.insert(children.end(), kids.begin(), kids.end());
        return id;
    }
};

thread_local std::string g_regex_error;

}  // namespace

struct wg_optree {
    Flat flat;
    int32_t root = 0;
};

extern "C" {

const char *wg_regex_error(void) { return g_regex_error.c_str(); }

namespace {
int32_t regex_to_optree(const char *pattern, int32_t length, bool fragment, wg_optree **out);
}

int32_t wg_regex_to_optree(const char *pattern, int32_t length, wg_optree **out) {
    return regex_to_optree(pattern, length, false, out);
}

namespace {
// fragment: the pattern is an argument that sits inside a larger output, so no end-of-sequence
// symbol follows it and its last repetition must be closed by the pattern itself.
int32_t regex_to_optree(const char *pattern, int32_t length, bool fragment, wg_optree **out) {
    if (!out) return WG_ERR_ARG;
    *out = nullptr;
    if (!pattern || length < 0 || length > (1 << 20)) return WG_ERR_ARG;
    g_regex_error.clear();
    try {
        std::vector<Re> arena;
        arena.reserve(4096);
        Parser ps{reinterpret_cast<const unsigned char *>(pattern), length, 0, arena};
        const int root = ps.parse_alt();
        if (ps.more()) ps.fail("unbalanced )");
        // the program is the pattern followed by the end-of-sequence symbol
        std::vector<int> items = {root};
        if (!fragment) {
            arena.push_back(Re{R_SET, Set{}, {}});
            arena.back().set.add(WG_SYM_EOS);
            items.push_back((int)arena.size() - 1);
        }
        Gen gen{arena};
        Chain chain;
        Set open = gen.gen(items, 0, Set{}, chain);
        if (!open.empty())
            throw Fail{fragment ? "a fragment must end with a character or class that closes its "
                                  "last repetition (the operators decide on the symbol that follows)"
                                : "internal: repetition left open at the end"};
        auto tree = std::make_unique<wg_optree>();
        tree->root = tree->flat.emit_chain(chain);
        if (tree->root < 0) throw Fail{"internal: empty program"};
        *out = tree.release();
        return WG_OK;
    } catch (const Fail &f) {
        g_regex_error = f.msg;
        return WG_ERR_GRAMMAR;
    } catch (const std::bad_alloc &) {
        g_regex_error = "out of memory";
        return WG_ERR_CAPACITY;
    }
}
}  // namespace

void wg_optree_free(wg_optree *tree) { delete tree; }

int32_t wg_optree_sizes(const wg_optree *tree, int32_t *n_nodes, int32_t *n_children,
                        int32_t *n_sets, int32_t *n_data, int32_t *root) {
    if (!tree) return WG_ERR_ARG;
    if (n_nodes) *n_nodes = (int32_t)tree->flat.nodes.size();
    if (n_children) *n_children = (int32_t)tree->flat.children.size();
    if (n_sets) *n_sets = (int32_t)(tree->flat.sets.size() / WG_SET_WORDS);
    if (n_data) *n_data = (int32_t)tree->flat.data.size();
    if (root) *root = tree->root;
    return WG_OK;
}

int32_t wg_optree_copy(const wg_optree *tree, wg_op_node *nodes, int32_t *children, uint32_t *sets,
                       uint8_t *data) {
    if (!tree) return WG_ERR_ARG;
    const Flat &f = tree->flat;
    if (nodes) memcpy(nodes, f.nodes.data(), f.nodes.size() * sizeof(wg_op_node));
    if (children && !f.children.empty()) memcpy(children, f.children.data(), f.children.size() * sizeof(int32_t));
    if (sets && !f.sets.empty()) memcpy(sets, f.sets.data(), f.sets.size() * sizeof(uint32_t));
    if (data && !f.data.empty()) memcpy(data, f.data.data(), f.data.size());
    return WG_OK;
}

namespace {
int32_t compile_regex(const char *pattern, int32_t length, bool fragment, wg_grammar **out);
}

int32_t wg_compile_regex(const char *pattern, int32_t length, wg_grammar **out) {
    return compile_regex(pattern, length, false, out);
}

int32_t wg_compile_regex_fragment(const char *pattern, int32_t length, wg_grammar **out) {
    return compile_regex(pattern, length, true, out);
}

namespace {
int32_t compile_regex(const char *pattern, int32_t length, bool fragment, wg_grammar **out) {
    if (!out) return WG_ERR_ARG;
    *out = nullptr;
    wg_optree *tree = nullptr;
    int32_t rc = regex_to_optree(pattern, length, fragment, &tree);
    if (rc != WG_OK) return rc;
    const Flat &f = tree->flat;
    rc = wg_compile_grammar(f.nodes.data(), (int32_t)f.nodes.size(), f.children.data(),
                            (int32_t)f.children.size(), f.sets.data(),
                            (int32_t)(f.sets.size() / WG_SET_WORDS), f.data.data(),
                            (int32_t)f.data.size(), tree->root, out);
    wg_optree_free(tree);
    return rc;
}
}  // namespace

}  // extern "C"
