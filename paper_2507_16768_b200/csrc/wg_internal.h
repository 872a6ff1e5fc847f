// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once

#include <cstdint>
#include <vector>

#include "wg.h"

constexpr int WG_N_SYMBOLS = 257;
constexpr int WG_SYM_EOS = 256;
constexpr int WG_SET_WORDS = 9;
constexpr int WG_REC_BYTES = 16;  // token bytes held in the fixed-size record

// A compiled grammar on the host: a dense table over byte classes.
// table[s * n_classes + c] is the state after any symbol of class c in state s; state 0 is
// DEAD (all of its entries are 0).  byte_class maps the 256 byte values, eos_class the EOS
// symbol.  Classes group symbols whose columns are equal in every state.
struct wg_grammar {
    int32_t n_states = 0;
    int32_t n_classes = 0;
    int32_t start = 0;
    int32_t done = 0;
    int32_t eos_class = 0;
    uint8_t byte_class[256] = {};
    std::vector<int32_t> table;
    // Token-level Write: forced_tok[s] >= 0 marks a state that accepts exactly that token id
    // (as a whole token) and continues in forced_next[s]; its table row is all DEAD.  Both
    // vectors are empty when the grammar has no such state.
    std::vector<int32_t> forced_tok, forced_next;
    // The state reached when the tree's own language is complete and only the implicit
    // end-of-sequence is still to come; -1 when the tree mentions EOS itself (there is no
    // implicit one then).  Splicing a grammar into a template redirects entries of this state.
    int32_t tail = -1;
    uint64_t hash = 0;
};

// One hole of a template: a placeholder state, the argument that fills it and the state
// where control continues once the argument's language is complete.
struct wg_hole_site {
    int32_t state, arg, next;
};

// A template (paper Section 3.1: a structure of the factory, parameterised but not yet
// instantiated): the table of its static part, with one placeholder state per hole.
struct wg_template {
    wg_grammar base;
    std::vector<wg_hole_site> sites;
    int32_t n_args = 0;
};

uint64_t wg_grammar_content_hash(const wg_grammar &g);

// Merges states with equal behaviour (wg_lower.cpp).  out may not alias in.
int32_t wg_minimize_grammar(const wg_grammar &in, wg_grammar *out);

// Lowering entry (wg_lower.cpp).
int32_t wg_lower_tree(const wg_op_node *nodes, int32_t n_nodes, const int32_t *children,
                      int32_t n_children, const uint32_t *sets, int32_t n_sets,
                      const uint8_t *data, int32_t n_data, int32_t root, wg_grammar *out,
                      std::vector<wg_hole_site> *sites = nullptr);

// Splices one compiled grammar per argument into the template's holes (wg_template.cpp).
int32_t wg_instantiate_template(const wg_template &t, const wg_grammar *const *args, int32_t n_args,
                                wg_grammar *out);
