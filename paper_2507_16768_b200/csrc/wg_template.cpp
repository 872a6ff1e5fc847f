// Template instantiation (paper Section 3.1: the frontend parser combines a request's
// arguments with the precompiled structure factory; contribution 2: the static structure is
// compiled offline, the dynamic arguments are injected at run time, composed from predefined
// grammar snippets).
//
// A template is a compiled table whose holes are placeholder states; an argument is a compiled
// grammar of its own.  Instantiation copies tables instead of lowering trees again: every hole
// site gets a private copy of its argument's states, entries of a placeholder are redirected to
// the copy's start state, and entries of the copy's tail state (the argument's language is
// complete) are redirected to the state that follows the hole.  The symbol classes of the result
// are the common refinement of the class maps involved.  Cost: one pass over the rows copied.
#include <cstring>
#include <vector>

#include "wg_internal.h"

namespace {

// Which arguments can be spliced: the tree must not have mentioned EOS (so it has a tail), and
// the tail must be what the lowering makes it: EOS leads to DONE, nothing else leaves it.
bool spliceable(const wg_grammar &g) {
    if (g.tail <= 0 || g.tail >= g.n_states || g.tail == g.done) return false;
    const int32_t *row = &g.table[(size_t)g.tail * g.n_classes];
    for (int32_t c = 0; c < g.n_classes; ++c)
        if (row[c] != (c == g.eos_class ? g.done : 0)) return false;
    return g.forced_tok.empty() || g.forced_tok[g.tail] < 0;
}

}  // namespace

int32_t wg_instantiate_template(const wg_template &t, const wg_grammar *const *args, int32_t n_args,
                                wg_grammar *out) {
    if (n_args != t.n_args || (n_args > 0 && !args)) return WG_ERR_ARG;
    for (int32_t a = 0; a < n_args; ++a) {
        if (!args[a]) return WG_ERR_ARG;
        if (!spliceable(*args[a])) return WG_ERR_GRAMMAR;
    }
    const wg_grammar &base = t.base;
    const int32_t n_sites = (int32_t)t.sites.size();

    // ---- joint symbol classes: refine the template's map by every distinct argument's map;
    // ids in order of first appearance over the symbols, as the lowering numbers them
    std::vector<int32_t> joint(WG_N_SYMBOLS);
    int32_t n_joint = 0;
    {
        std::vector<const wg_grammar *> parts{&base};
        for (int32_t a = 0; a < n_args; ++a) {
            bool seen = false;
            for (const wg_grammar *p : parts) seen |= p == args[a];
            if (!seen) parts.push_back(args[a]);
        }
        std::vector<int32_t> cur(WG_N_SYMBOLS, 0);
        int32_t n_cur = 1;
        std::vector<int32_t> renum;
        for (const wg_grammar *p : parts) {
            renum.assign((size_t)n_cur * p->n_classes, -1);
            int32_t n_next = 0;
            for (int sym = 0; sym < WG_N_SYMBOLS; ++sym) {
                const int32_t c = sym == WG_SYM_EOS ? p->eos_class : p->byte_class[sym];
                const size_t key = (size_t)cur[sym] * p->n_classes + c;
                if (renum[key] < 0) renum[key] = n_next++;
                cur[sym] = renum[key];
            }
            n_cur = n_next;
        }
        joint = cur;
        n_joint = n_cur;
    }
    if (n_joint > 256 + 1) return WG_ERR_ARG;  // cannot happen: there are 257 symbols
    std::vector<int32_t> rep(n_joint, -1);  // one representative symbol per joint class
    for (int sym = 0; sym < WG_N_SYMBOLS; ++sym)
        if (rep[joint[sym]] < 0) rep[joint[sym]] = sym;
    auto class_in = [](const wg_grammar &g, int sym) {
        return sym == WG_SYM_EOS ? g.eos_class : (int32_t)g.byte_class[sym];
    };

    // ---- state numbering: the template's states without the placeholders, then one block per
    // site holding the argument's states without DEAD, tail and DONE
    std::vector<int32_t> site_of(base.n_states, -1);
    for (int32_t i = 0; i < n_sites; ++i) {
        const wg_hole_site &h = t.sites[i];
        if (h.state <= 0 || h.state >= base.n_states || h.next <= 0 || h.next >= base.n_states ||
            h.arg < 0 || h.arg >= n_args || site_of[h.state] >= 0)
            return WG_ERR_ARG;
        site_of[h.state] = i;
    }
    std::vector<int32_t> t_id(base.n_states, -1);
    int32_t total = 0;
    for (int32_t s = 0; s < base.n_states; ++s)
        if (site_of[s] < 0) t_id[s] = total++;
    std::vector<int32_t> site_base(n_sites);
    // per argument: dense index of each of its states inside a site block (-1: not copied)
    std::vector<std::vector<int32_t>> arg_idx(n_args);
    std::vector<int32_t> arg_kept(n_args, 0);
    for (int32_t a = 0; a < n_args; ++a) {
        const wg_grammar &g = *args[a];
        arg_idx[a].assign(g.n_states, -1);
        int32_t n = 0;
        for (int32_t q = 1; q < g.n_states; ++q)
            if (q != g.tail && q != g.done) arg_idx[a][q] = n++;
        arg_kept[a] = n;
    }
    for (int32_t i = 0; i < n_sites; ++i) {
        site_base[i] = total;
        const int64_t next_total = (int64_t)total + arg_kept[t.sites[i].arg];
        if (next_total > 0x7FFFFFF0) return WG_ERR_CAPACITY;
        total = (int32_t)next_total;
    }
    // where a template state leads once the holes are filled: a placeholder stands for the
    // start of its argument's copy, or, for an argument that accepts only the empty string,
    // for whatever follows the hole (which may be the next hole)
    std::vector<int32_t> resolved(base.n_states, -1);
    for (int32_t s = 0; s < base.n_states; ++s) {
        int32_t at = s, hops = 0;
        while (site_of[at] >= 0) {
            const wg_hole_site &h = t.sites[site_of[at]];
            const wg_grammar &g = *args[h.arg];
            if (g.start != g.tail) break;
            at = h.next;
            if (++hops > n_sites) return WG_ERR_GRAMMAR;  // holes that only lead to each other
        }
        if (site_of[at] >= 0) {
            const wg_hole_site &h = t.sites[site_of[at]];
            resolved[s] = site_base[site_of[at]] + arg_idx[h.arg][args[h.arg]->start];
        } else {
            resolved[s] = t_id[at];
        }
    }

    const bool any_forced = [&] {
        if (!base.forced_tok.empty()) return true;
        for (int32_t a = 0; a < n_args; ++a)
            if (!args[a]->forced_tok.empty()) return true;
        return false;
    }();
    out->n_states = total;
    out->n_classes = n_joint;
    out->eos_class = joint[WG_SYM_EOS];
    for (int b = 0; b < 256; ++b) out->byte_class[b] = (uint8_t)joint[b];
    out->table.assign((size_t)total * n_joint, 0);
    out->forced_tok.clear();
    out->forced_next.clear();
    if (any_forced) {
        out->forced_tok.assign(total, -1);
        out->forced_next.assign(total, 0);
    }
    // ---- the template's rows
    {
        std::vector<int32_t> col(n_joint);
        for (int32_t c = 0; c < n_joint; ++c) col[c] = class_in(base, rep[c]);
        for (int32_t s = 1; s < base.n_states; ++s) {
            if (site_of[s] >= 0) continue;
            const int32_t *src = &base.table[(size_t)s * base.n_classes];
            int32_t *dst = &out->table[(size_t)t_id[s] * n_joint];
            for (int32_t c = 0; c < n_joint; ++c) dst[c] = resolved[src[col[c]]];
            if (!base.forced_tok.empty() && base.forced_tok[s] >= 0) {
                out->forced_tok[t_id[s]] = base.forced_tok[s];
                out->forced_next[t_id[s]] = resolved[base.forced_next[s]];
            }
        }
    }
    // ---- one copy of the argument's rows per site
    std::vector<int32_t> col(n_joint), target;
    for (int32_t i = 0; i < n_sites; ++i) {
        const wg_hole_site &h = t.sites[i];
        const wg_grammar &g = *args[h.arg];
        if (g.start == g.tail) continue;  // the empty string: nothing to copy
        for (int32_t c = 0; c < n_joint; ++c) col[c] = class_in(g, rep[c]);
        target.assign(g.n_states, 0);  // DEAD and DONE (reached from the tail only) map to DEAD
        for (int32_t q = 1; q < g.n_states; ++q)
            if (arg_idx[h.arg][q] >= 0) target[q] = site_base[i] + arg_idx[h.arg][q];
        target[g.tail] = resolved[h.next];
        for (int32_t q = 1; q < g.n_states; ++q) {
            if (arg_idx[h.arg][q] < 0) continue;
            const int32_t *src = &g.table[(size_t)q * g.n_classes];
            int32_t *dst = &out->table[(size_t)target[q] * n_joint];
            for (int32_t c = 0; c < n_joint; ++c) dst[c] = target[src[col[c]]];
            if (!g.forced_tok.empty() && g.forced_tok[q] >= 0) {
                out->forced_tok[target[q]] = g.forced_tok[q];
                out->forced_next[target[q]] = target[g.forced_next[q]];
            }
        }
    }
    out->start = resolved[base.start];
    out->done = t_id[base.done];
    out->tail = base.tail >= 0 ? resolved[base.tail] : -1;
    out->hash = wg_grammar_content_hash(*out);
    return WG_OK;
}
