/*
 * wg_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow CPU statement of what the allowed-token mask path computes, used only to
 * check the CUDA library: tests, the smoke entry and the CPU-baseline leg of the benchmark
 * call it; nothing in the product path does.  It shares no code, header, table or helper
 * with the library.
 *
 * Method (paper Section 3.2 and 3.3; operators Wait / Write / IfElse / DoWhile / Sequence):
 * the operator tree is INTERPRETED directly, one symbol at a time, with a cursor that names
 * the active primitive.  There is no transition table, no cache and no blocking.
 *
 * Alphabet: 257 symbols, bytes 0..255 and EOS = 256.  The end-of-sequence token is the
 * one-symbol string [EOS]; every other token is its byte string.
 *
 * Languages (A = allow, D = deny, W / T / F = wait, true_waits, false_waits,
 *            stay = (A \ D) \ (deciding symbols)):
 *   Write(b1..bn)                 exactly b1..bn            (Section 3.3: a chain of
 *                                                            single-element Waits)
 *   Wait(A, D, W, body)           stay* w L(body), w in W   (ends at the FIRST wait symbol:
 *                                                            non-greedy, Section 6)
 *   IfElse / Switch(cases Si)     stay* ( s_i L(body_i) )   (Section 3.2; absent body = empty)
 *   DoWhile(body, cond)           (L(body) stay* t)* L(body) stay* f   (Section 3.2 listing)
 *   Sequence(x1..xk)              concatenation
 *   WaitUntil(A, D, u, body)      the paper's Wait whose wait "token" is a multi-byte string u
 *                                 (Section 3.2: waits are tokens, e.g. a closing tag): any text
 *                                 over (A \ D) and the bytes of u, up to and including the FIRST
 *                                 occurrence of u, then L(body)
 *   WriteTokens(t1..tn)           the paper's own Write (Section 3.2: it emits a token sequence fixed
 *                                 in advance; Section 3.3: a chain of Waits each expecting one
 *                                 token): exactly these token ids, one per decode step.  It is
 *                                 entered and left only at token boundaries: no token's bytes
 *                                 may run into it or out of it.
 * Readings where the paper is silent: a tree in which no set mentions EOS is followed by an
 * implicit Wait(allow={EOS}, wait={EOS}); once the program has completed the cursor is DONE,
 * which accepts EOS only and stays DONE.
 *
 * Parity pins live in tests/ (the paper's worked example, closed forms, a regular-expression
 * library used as an independent partial matcher, brute force on tiny vocabularies).
 * Conventions the paper does not fix (bit order, the -inf patterns, k-way Switch, the
 * implicit EOS wait, byte-level Write) are "parity unpinned" by the paper itself and are
 * pinned only by those tests.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { K_SEQUENCE = 0, K_WRITE = 1, K_WAIT = 2, K_SWITCH = 3, K_DOWHILE = 4, K_WAIT_UNTIL = 5, K_WRITE_TOKENS = 6 };
enum { SYM_EOS = 256, SET_WORDS = 9 };
enum { CUR_DONE = -1, CUR_DEAD = -2, CUR_FINAL_EOS = -3 };
enum { ERR_ARG = -1, ERR_GRAMMAR = -2, ERR_REJECTED = -4 };

typedef struct {
    int32_t kind, n_child, child_off, n_set, set_off, data_off, data_len, reserved;
} node_t;

typedef struct wgo_tree {
    int32_t n_nodes, n_children, n_sets, n_data, root;
    node_t *nodes;
    int32_t *children;
    uint32_t *sets; /* [n_sets][9] */
    uint8_t *data;
    int32_t *parent; /* parent node of each node, -1 for the root */
    int32_t *slot;   /* position of the node in its parent's child list */
    int mentions_eos;
} wgo_tree;

typedef struct { int32_t node, off; } cursor_t;

static int in_set(const wgo_tree *t, int32_t set_index, int sym) {
    return (t->sets[(size_t)set_index * SET_WORDS + (sym >> 5)] >> (sym & 31)) & 1u;
}

static int set_empty(const wgo_tree *t, int32_t s) {
    for (int i = 0; i < SET_WORDS; i++) if (t->sets[(size_t)s * SET_WORDS + i]) return 0;
    return 1;
}

static int sets_meet(const wgo_tree *t, int32_t a, int32_t b) {
    for (int i = 0; i < SET_WORDS; i++)
        if (t->sets[(size_t)a * SET_WORDS + i] & t->sets[(size_t)b * SET_WORDS + i]) return 1;
    return 0;
}

void wgo_tree_free(wgo_tree *t) {
    if (!t) return;
    free(t->nodes); free(t->children); free(t->sets); free(t->data);
    free(t->parent); free(t->slot); free(t);
}

static void *dup_mem(const void *src, size_t bytes) {
    void *p = malloc(bytes ? bytes : 1);
    if (p && bytes) memcpy(p, src, bytes);
    return p;
}

/* Reads and validates the flat arrays.  Returns 0, ERR_ARG (malformed arrays) or
 * ERR_GRAMMAR (a well-formed tree the operator semantics reject). */
int wgo_tree_create(const int32_t *nodes, int32_t n_nodes, const int32_t *children,
                    int32_t n_children, const uint32_t *sets, int32_t n_sets,
                    const uint8_t *data, int32_t n_data, int32_t root, wgo_tree **out) {
    if (!out || n_nodes <= 0 || !nodes || root < 0 || root >= n_nodes) return ERR_ARG;
    if (n_children < 0 || n_sets < 0 || n_data < 0) return ERR_ARG;
    wgo_tree *t = (wgo_tree *)calloc(1, sizeof(wgo_tree));
    if (!t) return ERR_ARG;
    t->n_nodes = n_nodes; t->n_children = n_children; t->n_sets = n_sets; t->n_data = n_data;
    t->root = root;
    t->nodes = (node_t *)dup_mem(nodes, sizeof(node_t) * (size_t)n_nodes);
    t->children = (int32_t *)dup_mem(children, sizeof(int32_t) * (size_t)n_children);
    t->sets = (uint32_t *)dup_mem(sets, sizeof(uint32_t) * SET_WORDS * (size_t)n_sets);
    t->data = (uint8_t *)dup_mem(data, (size_t)n_data);
    t->parent = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_nodes);
    t->slot = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_nodes);
    int rc = 0;
    for (int i = 0; i < n_nodes; i++) { t->parent[i] = -2; t->slot[i] = 0; }
    t->parent[root] = -1;
    for (int i = 0; i < n_nodes && !rc; i++) {
        const node_t *n = &t->nodes[i];
        if (n->n_child < 0 || n->child_off < 0 || (int64_t)n->child_off + n->n_child > n_children ||
            n->n_set < 0 || n->set_off < 0 || (int64_t)n->set_off + n->n_set > n_sets ||
            n->data_len < 0 || n->data_off < 0 || (int64_t)n->data_off + n->data_len > n_data) {
            rc = ERR_ARG; break;
        }
        switch (n->kind) {
        case K_SEQUENCE: if (n->n_set != 0) rc = ERR_ARG; break;
        case K_WRITE: if (n->n_child != 0 || n->n_set != 0) rc = ERR_ARG; break;
        case K_WAIT: if (n->n_child != 1 || n->n_set != 3) rc = ERR_ARG; break;
        case K_SWITCH: if (n->n_set < 3 || n->n_child != n->n_set - 2) rc = ERR_ARG; break;
        case K_DOWHILE: if (n->n_child != 1 || n->n_set != 4) rc = ERR_ARG; break;
        case K_WAIT_UNTIL: if (n->n_child != 1 || n->n_set != 2) rc = ERR_ARG; break;
        case K_WRITE_TOKENS: if (n->n_child != 0 || n->n_set != 0 || n->data_len % 4) rc = ERR_ARG; break;
        default: rc = ERR_ARG;
        }
        if (rc) break;
        for (int j = 0; j < n->n_child; j++) {
            int32_t c = t->children[n->child_off + j];
            if (c == -1) {
                if (n->kind == K_SEQUENCE) rc = ERR_ARG; /* a Sequence part cannot be absent */
                continue;
            }
            if (c < 0 || c >= n_nodes) { rc = ERR_ARG; break; }
            if (t->parent[c] != -2) { rc = ERR_GRAMMAR; break; } /* shared or cyclic: not a tree */
            t->parent[c] = i; t->slot[c] = j;
        }
        if (rc) break;
        /* set rules: deciding sets non-empty, pairwise disjoint, disjoint from deny */
        if (n->kind == K_WAIT || n->kind == K_SWITCH || n->kind == K_DOWHILE) {
            int first = n->set_off + 2, last = n->set_off + n->n_set;
            for (int a = first; a < last && !rc; a++) {
                if (set_empty(t, a)) rc = ERR_GRAMMAR;
                if (sets_meet(t, a, n->set_off + 1)) rc = ERR_GRAMMAR;
                for (int b = a + 1; b < last && !rc; b++) if (sets_meet(t, a, b)) rc = ERR_GRAMMAR;
            }
        }
        if (n->kind == K_WAIT_UNTIL) { /* a non-empty string, none of whose bytes is denied */
            if (n->data_len < 1) rc = ERR_GRAMMAR;
            for (int j = 0; j < n->data_len && !rc; j++)
                if (in_set(t, n->set_off + 1, t->data[n->data_off + j])) rc = ERR_GRAMMAR;
        }
    }
    if (!rc) { /* every node must hang below the root exactly once */
        for (int i = 0; i < n_nodes; i++) if (t->parent[i] == -2) { rc = ERR_GRAMMAR; break; }
    }
    if (!rc) {
        for (int s = 0; s < n_sets; s++)
            if (t->sets[(size_t)s * SET_WORDS + 8] & 1u) t->mentions_eos = 1;
    }
    if (rc) { wgo_tree_free(t); return rc; }
    *out = t;
    return 0;
}

static cursor_t cur(int32_t node, int32_t off) { cursor_t c; c.node = node; c.off = off; return c; }

static cursor_t complete(const wgo_tree *t, int32_t n);

/* Descend to the first primitive of node n (an absent node is the empty string). */
static cursor_t enter(const wgo_tree *t, int32_t n, int32_t came_from) {
    if (n == -1) return complete(t, came_from);
    const node_t *nd = &t->nodes[n];
    switch (nd->kind) {
    case K_WRITE:
    case K_WRITE_TOKENS:
        return nd->data_len == 0 ? complete(t, n) : cur(n, 0);
    case K_WAIT:
    case K_SWITCH:
    case K_WAIT_UNTIL:
        return cur(n, 0);
    case K_DOWHILE: {
        int32_t body = t->children[nd->child_off];
        return body == -1 ? cur(n, 0) : enter(t, body, n);
    }
    default: /* K_SEQUENCE */
        return nd->n_child == 0 ? complete(t, n) : enter(t, t->children[nd->child_off], n);
    }
}

/* Node n has matched all of its language: what is active next? */
static cursor_t complete(const wgo_tree *t, int32_t n) {
    int32_t p = t->parent[n];
    if (p == -1) return t->mentions_eos ? cur(CUR_DONE, 0) : cur(CUR_FINAL_EOS, 0);
    const node_t *pd = &t->nodes[p];
    switch (pd->kind) {
    case K_SEQUENCE: {
        int32_t j = t->slot[n] + 1;
        return j < pd->n_child ? enter(t, t->children[pd->child_off + j], p) : complete(t, p);
    }
    case K_DOWHILE:
        return cur(p, 0); /* the body is done: the loop's condition is active */
    default: /* body of a Wait or of a Switch case */
        return complete(t, p);
    }
}

static cursor_t step(const wgo_tree *t, cursor_t c, int sym) {
    if (c.node == CUR_DEAD) return c;
    if (c.node == CUR_DONE || c.node == CUR_FINAL_EOS)
        return sym == SYM_EOS ? cur(CUR_DONE, 0) : cur(CUR_DEAD, 0);
    const node_t *nd = &t->nodes[c.node];
    if (nd->kind == K_WRITE_TOKENS) return cur(CUR_DEAD, 0); /* only whole tokens pass here */
    if (nd->kind == K_WRITE) {
        if (sym >= 256 || t->data[nd->data_off + c.off] != (uint8_t)sym) return cur(CUR_DEAD, 0);
        return c.off + 1 == nd->data_len ? complete(t, c.node) : cur(c.node, c.off + 1);
    }
    int32_t allow = nd->set_off, deny = nd->set_off + 1;
    if (nd->kind == K_WAIT_UNTIL) {
        /* c.off = how many bytes of u the text read so far ends with (the longest such
         * prefix of u).  After one more symbol: the longest prefix of u that is a suffix of
         * u[0..off) + symbol, found by trying every length from the top. */
        const uint8_t *u = t->data + nd->data_off;
        const int len = nd->data_len;
        int is_u_byte = 0;
        for (int j = 0; j < len; j++) if (sym < 256 && u[j] == (uint8_t)sym) is_u_byte = 1;
        if (!is_u_byte && !(in_set(t, allow, sym) && !in_set(t, deny, sym))) return cur(CUR_DEAD, 0);
        if (sym >= 256) return cur(c.node, 0); /* EOS is never part of u */
        int best = 0;
        for (int j = (c.off + 1 < len ? c.off + 1 : len); j >= 1 && !best; j--) {
            /* does u[0..j) equal the last j symbols of u[0..off) + symbol? */
            int same = u[j - 1] == (uint8_t)sym;
            for (int i = 0; i < j - 1 && same; i++)
                if (u[i] != u[c.off - (j - 1) + i]) same = 0;
            if (same) best = j;
        }
        if (best == len) return enter(t, t->children[nd->child_off], c.node);
        return cur(c.node, best);
    }
    if (nd->kind == K_WAIT) {
        if (in_set(t, nd->set_off + 2, sym)) return enter(t, t->children[nd->child_off], c.node);
    } else if (nd->kind == K_SWITCH) {
        for (int i = 0; i < nd->n_child; i++)
            if (in_set(t, nd->set_off + 2 + i, sym))
                return enter(t, t->children[nd->child_off + i], c.node);
    } else { /* condition of a DoWhile */
        if (in_set(t, nd->set_off + 2, sym)) { /* true: run the body again */
            int32_t body = t->children[nd->child_off];
            return body == -1 ? c : enter(t, body, c.node);
        }
        if (in_set(t, nd->set_off + 3, sym)) return complete(t, c.node);
    }
    if (in_set(t, allow, sym) && !in_set(t, deny, sym)) return c; /* stay */
    return cur(CUR_DEAD, 0);
}

void wgo_start(const wgo_tree *t, int32_t *out) {
    cursor_t c = enter(t, t->root, -1);
    out[0] = c.node; out[1] = c.off;
}

void wgo_step(const wgo_tree *t, const int32_t *in, int32_t sym, int32_t *out) {
    cursor_t c = step(t, cur(in[0], in[1]), sym);
    out[0] = c.node; out[1] = c.off;
}

/* Token t from cursor c: the cursor after its symbols, DEAD if any symbol is refused.
 * A zero-length token other than EOS is refused (it would leave the request where it is). */
static cursor_t walk_token(const wgo_tree *t, cursor_t c, const uint32_t *offsets,
                           const uint8_t *bytes, int32_t eos_id, int32_t tok) {
    if (c.node >= 0 && t->nodes[c.node].kind == K_WRITE_TOKENS) {
        /* the next token of the forced sequence, as a whole token, and nothing else */
        const node_t *nd = &t->nodes[c.node];
        int32_t want;
        memcpy(&want, t->data + nd->data_off + 4 * c.off, 4);
        if (tok != want) return cur(CUR_DEAD, 0);
        return 4 * (c.off + 1) == nd->data_len ? complete(t, c.node) : cur(c.node, c.off + 1);
    }
    if (tok == eos_id) return step(t, c, SYM_EOS);
    uint32_t b = offsets[tok], e = offsets[tok + 1];
    if (b == e) return cur(CUR_DEAD, 0);
    for (uint32_t i = b; i < e && c.node != CUR_DEAD; i++) c = step(t, c, bytes[i]);
    return c;
}

/* Mask of one cursor: bit (t & 31) of word (t >> 5) is 1 iff token t is allowed.
 * Bits at and beyond V in the last word are 0. */
void wgo_mask(const wgo_tree *t, const uint32_t *offsets, const uint8_t *bytes, int32_t V,
              int32_t eos_id, const int32_t *cursor, uint32_t *words) {
    int32_t W = (V + 31) / 32;
    memset(words, 0, sizeof(uint32_t) * (size_t)W);
    cursor_t c = cur(cursor[0], cursor[1]);
    for (int32_t tok = 0; tok < V; tok++) {
        cursor_t r = walk_token(t, c, offsets, bytes, eos_id, tok);
        if (r.node != CUR_DEAD) words[tok >> 5] |= 1u << (tok & 31);
    }
}

/* One mask per row; trees[r] and cursors[2r..2r+1] belong to row r.  Rows are independent,
 * so threads (when asked for) simply take different rows. */
void wgo_masks(const wgo_tree *const *trees, const uint32_t *offsets, const uint8_t *bytes,
               int32_t V, int32_t eos_id, const int32_t *cursors, int32_t B, uint32_t *out,
               int64_t row_stride_words, int32_t n_threads) {
    (void)n_threads;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(n_threads > 0 ? n_threads : 1)
#endif
    for (int32_t r = 0; r < B; r++)
        wgo_mask(trees[r], offsets, bytes, V, eos_id, cursors + 2 * r, out + r * row_stride_words);
}

/* Apply: every token whose bit is clear gets the -inf pattern; all other elements keep
 * their bits.  Works on raw bit patterns (fp32: 0xFF800000, bf16: 0xFF80). */
void wgo_apply_f32(uint32_t *logits, int64_t row_stride, const uint32_t *mask,
                   int64_t mask_stride, int32_t B, int32_t V, int32_t n_threads) {
    (void)n_threads;
#ifdef _OPENMP
#pragma omp parallel for num_threads(n_threads > 0 ? n_threads : 1)
#endif
    for (int32_t r = 0; r < B; r++)
        for (int32_t tok = 0; tok < V; tok++)
            if (!((mask[r * mask_stride + (tok >> 5)] >> (tok & 31)) & 1u))
                logits[r * row_stride + tok] = 0xFF800000u;
}

void wgo_apply_bf16(uint16_t *logits, int64_t row_stride, const uint32_t *mask,
                    int64_t mask_stride, int32_t B, int32_t V, int32_t n_threads) {
    (void)n_threads;
#ifdef _OPENMP
#pragma omp parallel for num_threads(n_threads > 0 ? n_threads : 1)
#endif
    for (int32_t r = 0; r < B; r++)
        for (int32_t tok = 0; tok < V; tok++)
            if (!((mask[r * mask_stride + (tok >> 5)] >> (tok & 31)) & 1u))
                logits[r * row_stride + tok] = 0xFF80u;
}

static float bits_to_float(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* Greedy choice: scan allowed tokens in ascending id and replace the best on a strict '>',
 * so the lowest id among equal maxima wins and -0.0 ties with +0.0.  No allowed token: -1. */
void wgo_argmax_f32(const uint32_t *logits, int64_t row_stride, const uint32_t *mask,
                    int64_t mask_stride, int32_t B, int32_t V, int32_t *out) {
    for (int32_t r = 0; r < B; r++) {
        int32_t best = -1; float bv = 0.0f;
        for (int32_t tok = 0; tok < V; tok++) {
            if (!((mask[r * mask_stride + (tok >> 5)] >> (tok & 31)) & 1u)) continue;
            float v = bits_to_float(logits[r * row_stride + tok]);
            if (best < 0 || v > bv) { best = tok; bv = v; }
        }
        out[r] = best;
    }
}

void wgo_argmax_bf16(const uint16_t *logits, int64_t row_stride, const uint32_t *mask,
                     int64_t mask_stride, int32_t B, int32_t V, int32_t *out) {
    for (int32_t r = 0; r < B; r++) {
        int32_t best = -1; float bv = 0.0f;
        for (int32_t tok = 0; tok < V; tok++) {
            if (!((mask[r * mask_stride + (tok >> 5)] >> (tok & 31)) & 1u)) continue;
            float v = bits_to_float((uint32_t)logits[r * row_stride + tok] << 16); /* exact */
            if (best < 0 || v > bv) { best = tok; bv = v; }
        }
        out[r] = best;
    }
}

/* Advance: the cursor after the chosen token; a refused token (or an id outside 0..V-1)
 * leaves the cursor unchanged and returns ERR_REJECTED. */
int wgo_advance(const wgo_tree *t, const uint32_t *offsets, const uint8_t *bytes, int32_t V,
                int32_t eos_id, int32_t *cursor, int32_t token) {
    if (token < 0 || token >= V) return ERR_REJECTED;
    cursor_t r = walk_token(t, cur(cursor[0], cursor[1]), offsets, bytes, eos_id, token);
    if (r.node == CUR_DEAD) return ERR_REJECTED;
    cursor[0] = r.node; cursor[1] = r.off;
    return 0;
}

int wgo_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
