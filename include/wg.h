/*
 * wg.h -- C ABI of the allowed-token mask path for operator-automaton structured decoding.
 *
 * What the path computes (paper Section 1: the mask is a vocabulary-sized binary tensor,
 * ones = allowed, applied to the logits before sampling; Section 3.2: Wait / Write / IfElse /
 * DoWhile / Sequence operators tracked by a finite state machine, one transition per
 * generated token; Section 3.3: masks depend on the operator state only, so they are cached
 * globally across steps and requests):
 *
 *   for every request r of a batch, with grammar id gid[r] and automaton state sid[r]:
 *     bitmask[r, t>>5] bit (t&31) = 1  iff  the bytes of token t, walked from sid[r] through
 *                                       the grammar's byte-level transition table, never
 *                                       reach the DEAD state           (wg_build_masks)
 *     masks of states seen before are served from a device cache       (wg_mask_cache_lookup)
 *     logits[r, t] = -inf where the bit is clear, in place             (wg_apply_mask)
 *     optionally token[r] = lowest id among the maxima of the allowed logits
 *     sid[r] = state after the chosen token's bytes                    (wg_advance)
 *
 * Conventions
 *   - Every call returns WG_OK (0) or a negative wg_status.  Nothing aborts or throws.
 *   - "host" pointers are read during the call and may be freed afterwards.  "device"
 *     pointers are owned by the caller, must belong to the CUDA device that was current when
 *     the wg_ctx was created, and must stay valid until the work queued on `stream` is done.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Device
 *     calls only enqueue work; they do not synchronise unless stated.
 *   - A wg_ctx keeps per-call scratch: calls on one context must be issued from one thread at
 *     a time and on one stream at a time (or on streams ordered by events).  Use one context
 *     per concurrent stream; vocabularies and compiled grammars may be shared between them.
 *   - Every object belongs to the CUDA device that was current when it was created; make
 *     that device current before calling into it.
 *   - The cache never evicts: when its pool is full, further new states are built straight
 *     into the caller's bitmask on every step (counted as rows_uncached) until
 *     wg_cache_clear is called.
 *   - Per-row problems found on the device (a refused token, an empty mask, an unknown
 *     state) are written to the optional per-row status array and counted in wg_stats; they
 *     never fault the GPU.
 *   - Alphabet: symbols 0..255 are byte values, symbol 256 is end-of-sequence (EOS).  The EOS
 *     token (id `eos_id`) stands for the one-symbol string [EOS]; any other token is its byte
 *     string.  A zero-length token other than EOS is never allowed.
 *   - State 0 of every compiled grammar is DEAD.  State ids are dense, 0 .. n_states-1.
 *   - Packed masks: uint32 words, bit (t & 31) of word (t >> 5) belongs to token t, 1 =
 *     allowed, bits at and beyond V are 0.  W = ceil(V / 32) words per row.
 */
#ifndef WG_H_
#define WG_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum wg_status {
    WG_OK = 0,
    WG_ERR_ARG = -1,            /* null pointer, bad size, bad stride, unknown id            */
    WG_ERR_GRAMMAR = -2,        /* the operator tree breaks a rule listed at wg_compile_grammar */
    WG_ERR_CAPACITY = -3,       /* a fixed-size table of the library is full                 */
    WG_ERR_TOKEN_REJECTED = -4, /* per row: the token is not allowed in the row's state      */
    WG_ERR_CUDA = -5,           /* a CUDA runtime call failed; see wg_last_cuda_error        */
    WG_ERR_EMPTY_MASK = -6,     /* per row: no token is allowed, so there is no argmax       */
    WG_ERR_STATE = -7           /* per row: grammar id or state id out of range              */
} wg_status;

/* Most rows one call may take: the row number is the second grid dimension of the apply
 * kernels.  wg_ctx_create refuses a larger max_batch, wg_apply_mask a larger B (WG_ERR_ARG). */
#define WG_MAX_ROWS 65535

/* Logit element types of wg_apply_mask / wg_decode_step. */
enum { WG_DTYPE_BF16 = 0, WG_DTYPE_FP32 = 1 };

/* Flags of wg_build_masks and wg_decode_step. */
enum {
    WG_USE_CACHE = 0u, /* look up (gid, sid); build and insert the misses; copy rows out   */
    WG_NO_CACHE = 1u   /* build every row, duplicates included; the cache is not touched   */
};

/* Flags of wg_advance and wg_decode_step. */
enum {
    WG_RESTART_ON_DONE = 2u /* a row that reaches the DONE state starts over at the grammar's
                               start state (a finished request is replaced by a new one)   */
};

/* Operator kinds of wg_op_node (paper Section 3.2). */
enum {
    WG_OP_SEQUENCE = 0,
    WG_OP_WRITE = 1,
    WG_OP_WAIT = 2,
    WG_OP_SWITCH = 3, /* IfElse and its k-way generalisation */
    WG_OP_DOWHILE = 4,
    WG_OP_WAIT_UNTIL = 5,  /* a Wait whose wait "token" is a multi-byte string */
    WG_OP_WRITE_TOKENS = 6, /* the paper's token-level Write: forced token ids       */
    WG_OP_HOLE = 7          /* templates only: the place of a run-time argument      */
};

/* One node of a flattened operator tree.  Children, symbol sets and literal bytes live in
 * three side arrays; a node names its slice of each.  A symbol set is 9 uint32 words, bit
 * (s & 31) of word (s >> 5) for symbol s, symbol 256 = EOS.
 *   SEQUENCE  children = the parts, in order
 *   WRITE     data     = the literal bytes
 *   WAIT      sets     = [allow, deny, wait],               children = [body or -1]
 *   SWITCH    sets     = [allow, deny, case_0 .. case_k-1], children = [body_0 .. body_k-1]
 *             (IfElse: case_0 = true_waits -> if_body, case_1 = false_waits -> else_body)
 *   DOWHILE   sets     = [allow, deny, true_waits, false_waits], children = [body or -1]
 *   WAIT_UNTIL sets    = [allow, deny], data = the string waited for, children = [body or -1]
 *             (paper Section 3.2: the waits of a Wait are tokens, e.g. a closing tag; at byte
 *             level such a token is a string.  Accepts text over (allow \ deny) and the
 *             string's own bytes up to and including the FIRST occurrence of the string.)
 *   WRITE_TOKENS data  = the forced token ids, 4 little-endian bytes each (ids >= 0)
 *             (paper Section 3.2: Write emits a token sequence fixed in advance; Section 3.3:
 *             a chain of Waits each expecting one token.  Exactly these ids, one per decode
 *             step; entered and left at token boundaries only, so no token's bytes may run
 *             into or out of it.  An id beyond the vocabulary yields an empty mask.)
 *   HOLE      reserved = index of the argument that fills it (wg_template_compile only) */
typedef struct wg_op_node {
    int32_t kind;
    int32_t n_child, child_off;
    int32_t n_set, set_off;
    int32_t data_off, data_len;
    int32_t reserved;
} wg_op_node;

typedef struct wg_vocab wg_vocab;     /* token byte strings, resident on one device */
typedef struct wg_grammar wg_grammar; /* a compiled transition table, host side     */
typedef struct wg_ctx wg_ctx;         /* device tables, mask cache and scratch      */

/* Storage of the mask cache (wg_ctx_create_ex) and the two forms of a compact entry. */
enum {
    WG_CACHE_DENSE = 0,  /* one packed mask row of W words per cached state                    */
    WG_CACHE_COMPACT = 1 /* adaptive allows / denies entries (paper Section 3.3)               */
};
enum {
    WG_ENTRY_ALLOWS = 0, /* reject-heavy state: the entry keeps the allowed tokens             */
    WG_ENTRY_DENIES = 1  /* accept-heavy state: the entry keeps the refused tokens             */
};

typedef struct wg_stats {
    int64_t cache_hits;      /* rows served from the cache                                  */
    int64_t cache_misses;    /* rows whose mask had to be built (first sight of the state)  */
    int64_t masks_built;     /* masks produced by the build kernel                          */
    int64_t rows_uncached;   /* rows built outside the cache because it was full            */
    int64_t tokens_rejected; /* rows of wg_advance whose token was refused                  */
    int64_t empty_masks;     /* rows whose argmax found no allowed token                    */
    int64_t bad_states;      /* rows with a grammar or state id out of range                */
    int64_t cache_entries;   /* states held by the cache now                                */
    int64_t cache_bytes;     /* device memory those cached masks occupy                     */
} wg_stats;

/* ---- setup ------------------------------------------------------------------------- */

/* Copies a vocabulary to the current device.  The tokens are given in CSR form (paper
 * Section 3.1 keeps a token-to-id map in the structure factory; here the map is the byte
 * string of every id): token t is bytes[offsets[t] .. offsets[t+1]).
 *   offsets  host, V + 1 entries, non-decreasing, offsets[0] = 0
 *   bytes    host, offsets[V] bytes (may be NULL when that is 0)
 *   eos_id   0 <= eos_id < V; the bytes given for it are ignored
 * The library keeps its own device copy: the first 16 bytes of every token in fixed-size
 * records, the lengths, and the CSR arrays for longer tokens.  Free with wg_vocab_free.
 * Errors: WG_ERR_ARG (null, V <= 0, bad offsets, eos_id out of range), WG_ERR_CUDA. */
int32_t wg_load_vocab(const uint32_t *offsets, const uint8_t *bytes, int32_t V, int32_t eos_id,
                      wg_vocab **out);
void wg_vocab_free(wg_vocab *vocab);

/* Lowers an operator tree to a byte-level deterministic transition table, on the host
 * (paper Section 3.2: operator composition; the paper tracks operators per token, this
 * library walks token BYTES, so a literal may be produced by any tokens whose bytes spell it).
 * All pointers are host arrays in the layout described at wg_op_node.
 * Languages: Write = its literal; Wait = stay* w body (ends at the first wait symbol, paper
 * Section 6); WaitUntil = text up to the first occurrence of its string, then body; Switch = stay* (s_i body_i); DoWhile = (body stay* t)* body stay* f; Sequence =
 * concatenation; stay = (allow \ deny) \ deciding symbols; an absent body is empty.  If no
 * set mentions EOS, the program is followed by one EOS.  After the program comes the DONE
 * state, which accepts EOS only and stays DONE.
 * Errors: WG_ERR_ARG for malformed arrays; WG_ERR_GRAMMAR for an empty deciding set,
 * deciding sets that overlap each other or the deny set, an empty or partly denied WaitUntil
 * string, or a node used twice (not a tree). */
int32_t wg_compile_grammar(const wg_op_node *nodes, int32_t n_nodes, const int32_t *children,
                           int32_t n_children, const uint32_t *sets, int32_t n_sets,
                           const uint8_t *data, int32_t n_data, int32_t root, wg_grammar **out);
void wg_grammar_free(wg_grammar *grammar);

/* Regular-expression front end (paper Section 3.2, the paragraph on translating regular
 * expressions into Wait / Write compositions; the syntax-prior variant evaluated in Section 4.1).
 * Translates a pattern into an operator tree: classes and characters become Wait, literal runs
 * Write, repetition and branching DoWhile / IfElse(Switch) / Sequence, followed by EOS.
 * Dialect (bytes): literals, '.', escapes \d \w \s \D \W \S \n \t \r \f \v \0 \xHH
 * and \<punctuation>, classes [a-z0-9_] and [^...], groups ( ) and (?: ), '|', and the
 * quantifiers * + ? {m} {m,} {m,n} (n <= 64; a trailing lazy '?' is ignored).  '^' at the very
 * start and '$' at the very end are accepted and mean nothing: the whole output must match.
 * The operators decide on one symbol, so wherever the pattern chooses (stay in a repetition
 * or leave it, which alternative) the candidate first symbols must not overlap, a repeated
 * group must begin with a character, class or repeated class, and what follows a repetition
 * must begin with one as well.  Anything else returns WG_ERR_GRAMMAR; wg_regex_error() then
 * gives the reason (thread-local, valid until the next call on the thread).
 *   pattern  host, `length` bytes, need not be NUL-terminated
 * wg_compile_regex = wg_regex_to_optree + wg_compile_grammar.  The tree itself can be read
 * back with wg_optree_sizes / wg_optree_copy (arrays as in wg_compile_grammar; any pointer of
 * wg_optree_copy may be NULL to skip that array).  Free with wg_optree_free. */
typedef struct wg_optree wg_optree;
int32_t wg_regex_to_optree(const char *pattern, int32_t length, wg_optree **out);
int32_t wg_optree_sizes(const wg_optree *tree, int32_t *n_nodes, int32_t *n_children,
                        int32_t *n_sets, int32_t *n_data, int32_t *root);
int32_t wg_optree_copy(const wg_optree *tree, wg_op_node *nodes, int32_t *children, uint32_t *sets,
                       uint8_t *data);
void wg_optree_free(wg_optree *tree);
int32_t wg_compile_regex(const char *pattern, int32_t length, wg_grammar **out);
/* The same for a pattern that is an ARGUMENT of a template (wg_template_instantiate): no EOS
 * follows it, and because the operators decide on the symbol that follows a repetition, the
 * pattern itself must close its last repetition (`[0-9]+"` is a fragment, `[0-9]+` is not:
 * WG_ERR_GRAMMAR). */
int32_t wg_compile_regex_fragment(const char *pattern, int32_t length, wg_grammar **out);
const char *wg_regex_error(void);

/* Templates: the static part of a structure compiled once, arguments spliced in per request
 * (paper Section 3.1: the structure factory holds structures that are parameterised but not yet
 * instantiated, and a request's arguments are combined with it into the request's state
 * machine; contribution 2: static structure precompiled offline, dynamic arguments injected at
 * run time and composed from predefined grammar snippets).
 * wg_template_compile lowers an operator tree that may contain HOLE nodes (arrays as in
 *   wg_compile_grammar); the same argument index may occur at several holes.
 * wg_template_instantiate fills every hole with a compiled grammar -- args[i] for the holes
 *   of argument i -- by copying table rows, without lowering anything again: a hole's entries
 *   lead to the start of a private copy of the argument's states, and where the argument's
 *   language is complete control continues after the hole.  The result is an ordinary grammar
 *   whose language is that of the tree with each hole replaced by its argument's tree.  An
 *   argument must be compiled from a tree that mentions EOS in no set (arguments sit inside
 *   the output, they do not end it); anything else gives WG_ERR_GRAMMAR.  Argument grammars
 *   can be compiled once and reused across requests and holes (predefined snippets), come from
 *   wg_compile_regex, or be loaded from blobs.  Cost: proportional to the rows copied
 *   (states x symbol classes), typically a small fraction of lowering the whole tree.
 * Errors: WG_ERR_ARG (null, n_args different from the template's, malformed arrays),
 *   WG_ERR_GRAMMAR, WG_ERR_CAPACITY. */
typedef struct wg_template wg_template;
int32_t wg_template_compile(const wg_op_node *nodes, int32_t n_nodes, const int32_t *children,
                            int32_t n_children, const uint32_t *sets, int32_t n_sets,
                            const uint8_t *data, int32_t n_data, int32_t root, wg_template **out);
/* n_states counts the template's own states (placeholders included); n_holes the hole sites
 * that can be reached; n_args = 1 + the largest argument index.  Any pointer may be NULL. */
int32_t wg_template_info(const wg_template *tmpl, int32_t *n_states, int32_t *n_holes,
                         int32_t *n_args);
int32_t wg_template_instantiate(const wg_template *tmpl, const wg_grammar *const *args,
                                int32_t n_args, wg_grammar **out);
void wg_template_free(wg_template *tmpl);

/* Returns in *out a grammar with the same language in which states that behave alike are
 * merged (classical DFA minimisation by partition refinement).  The paper caches masks per
 * operator state (Section 3.3); merged states share one cached mask, and grammars that
 * repeat a tail (enum entries with a common ending, the tails a regular expression's
 * alternatives carry) shrink a lot.  State ids change: states taken from the input grammar
 * do not carry over.  Host side; cost about n_states * n_classes * log(n_states) per round of
 * refinement.  The input is left as it is; free both. */
int32_t wg_grammar_minimize(const wg_grammar *grammar, wg_grammar **out);

/* A compiled grammar as a flat byte blob, so that tables compiled offline can be stored and
 * loaded at start-up instead of being recompiled (paper Section 3.1: the static structure is
 * processed once, offline, into an artefact that requests reuse).
 * wg_grammar_save: writes at most `capacity` bytes to `blob` and always stores the size the
 *   blob needs in *needed; returns WG_ERR_CAPACITY (nothing written) if capacity is too
 *   small, so a first call with blob = NULL, capacity = 0 asks for the size.
 * wg_grammar_load: rebuilds a grammar from such a blob after checking it (magic, version,
 *   sizes, every table entry and state id in range, and the stored content hash against the
 *   hash of what was read); a damaged blob gives WG_ERR_ARG.
 * The format is little-endian and private to this library version. */
int32_t wg_grammar_save(const wg_grammar *grammar, void *blob, size_t capacity, size_t *needed);
int32_t wg_grammar_load(const void *blob, size_t size, wg_grammar **out);

/* Host-side facts about a compiled grammar.  Any output pointer may be NULL.
 * content_hash identifies the table: two compilations with equal tables hash equally. */
int32_t wg_grammar_info(const wg_grammar *grammar, int32_t *n_states, int32_t *start_state,
                        int32_t *done_state, int32_t *n_classes, uint64_t *content_hash);

/* Host-side single transition: the state after `symbol` (0..256) in `state`, 0 = DEAD.
 * Out-of-range arguments give 0.  For tests and tooling; not on the decode path. */
int32_t wg_grammar_step(const wg_grammar *grammar, int32_t state, int32_t symbol);

/* Host-side: is `state` a forced-token state of a WRITE_TOKENS operator?  Returns 1 and fills
 * *token / *next_state (either may be NULL) if so, 0 otherwise (also for bad arguments). */
int32_t wg_grammar_forced_token(const wg_grammar *grammar, int32_t state, int32_t *token,
                                int32_t *next_state);

/* Creates the device context on the current device: grammar table registry, the mask cache
 * (a hash table keyed by (grammar id, state id) plus a pool of `cache_capacity` mask rows,
 * paper Section 3.3) and per-batch scratch for up to `max_batch` rows per call.
 * cache_capacity may be 0 (every WG_USE_CACHE row is then built uncached).  max_batch <= WG_MAX_ROWS.
 * The vocabulary must outlive the context.  Errors: WG_ERR_ARG, WG_ERR_CUDA. */
int32_t wg_ctx_create(const wg_vocab *vocab, int32_t cache_capacity, int32_t max_batch,
                      wg_ctx **out);
void wg_ctx_free(wg_ctx *ctx);

/* wg_ctx_create with a choice of cache storage.
 * WG_CACHE_DENSE is wg_ctx_create.  WG_CACHE_COMPACT stores every cached mask the way the
 * paper's Wait operator keeps its token sets (Section 3.3: a few refused tokens in `denies`
 * when most of the vocabulary is accepted, the accepted ones in `allows` when most is
 * refused): the side with fewer tokens is kept.  On the device the choice is made for every
 * span of 1024 tokens by itself (never worse than one choice per mask), and a span holds its
 * listed tokens grouped by 32-token mask word: only the words that contain a listed token are
 * stored, behind an 8-byte header per span, so a mask never takes more room than its id list
 * plus the headers, and a row is masked straight from it.  Masks of literal states and of
 * free-text slots shrink from V/8 bytes to about a kilobyte, which is what lets grammars with
 * hundreds of thousands of states stay cached.  Results of every call are identical in both
 * modes; wg_cache_entry_read reports an entry as the paper's per-mask allows / denies set.
 *   arena_bytes  device memory for the stored words; 0 = a quarter of what cache_capacity
 *                dense rows would take (the span headers, capacity x ceil(W/32) x 8 bytes,
 *                come on top).  When the arena is full, further new states are built on
 *                every step (counted as rows_uncached), as with a full dense pool.
 * Errors: WG_ERR_ARG (also: unknown cache_mode), WG_ERR_CUDA. */
int32_t wg_ctx_create_ex(const wg_vocab *vocab, int32_t cache_capacity, int32_t max_batch,
                         int32_t cache_mode, size_t arena_bytes, wg_ctx **out);

/* Reads one cached entry of a WG_CACHE_COMPACT context back to the host as the paper's token
 * set: *kind = WG_ENTRY_ALLOWS or WG_ENTRY_DENIES (or -1 when (grammar_id, state) is not
 * cached), *n_listed = number of tokens on the kept side, ids_host[0 .. min(n_listed,
 * ids_capacity)) = those token ids in ascending order, *entry_bytes = device bytes the entry
 * occupies.  Any output pointer may be NULL.  For tests and tooling; synchronises `stream`.
 * Errors: WG_ERR_ARG (also for a dense context), WG_ERR_CUDA. */
int32_t wg_cache_entry_read(wg_ctx *ctx, int32_t grammar_id, int32_t state, int32_t *kind,
                            int32_t *n_listed, int32_t *ids_host, int32_t ids_capacity,
                            int64_t *entry_bytes, void *stream);

/* Uploads a compiled grammar's table and returns its id in this context.  A grammar whose
 * content_hash, tables, symbol-class map and start / DONE states all equal those of one
 * already added gets that grammar's id, so requests
 * instantiated with the same arguments share cache entries.  Synchronous: the table is
 * copied and a few set-up kernels run on the legacy default stream, which the call waits for
 * (so it must not be made while a stream capture is under way).
 * The id may be one that wg_ctx_remove_grammar set free.
 * Errors: WG_ERR_ARG, WG_ERR_CAPACITY (more than 65535 grammars at a time, or a table of 2^32
 * cells or more), WG_ERR_CUDA. */
int32_t wg_ctx_add_grammar(wg_ctx *ctx, const wg_grammar *grammar, int32_t *grammar_id);

/* Takes grammar `grammar_id` out of the context again (paper Section 3.1: a state machine is
 * made per request from the request's arguments, so a serving process adds grammars for as long
 * as it runs).  The grammar's device tables are freed, its cached masks stop matching and their
 * pool rows are handed out to later states (the words a compact entry took in the arena come
 * back only with wg_cache_clear), and the id is given to a grammar added later -- at most 65535
 * grammars are held AT A TIME.  From the call on, a row that still names the id is treated as a
 * row in a state the grammar does not have: an all-zero mask, WG_ERR_STATE, bad_states counted.
 * Synchronous: waits for everything queued on the device first (no stream capture may be under
 * way); a step recorded with wg_step_graph_create for rows of this grammar must not be launched
 * afterwards.  When removed entries hold a quarter of the hash table it is rebuilt without them.
 * Errors: WG_ERR_ARG (no such grammar), WG_ERR_CUDA. */
int32_t wg_ctx_remove_grammar(wg_ctx *ctx, int32_t grammar_id);

/* Builds and caches the mask of every state of grammar `grammar_id` (states 1..n_states-1),
 * max_batch states at a time.  Returns WG_ERR_CAPACITY after the first batch that found the
 * pool (or the arena) full; the states cached up to then stay cached.  Synchronises `stream`
 * after every batch. */
int32_t wg_cache_prewarm(wg_ctx *ctx, int32_t grammar_id, void *stream);

/* Forgets every cached mask (enqueued on `stream`). */
int32_t wg_cache_clear(wg_ctx *ctx, void *stream);

/* Copies the device counters to *out.  Synchronises `stream`. */
int32_t wg_get_stats(wg_ctx *ctx, wg_stats *out, void *stream);
int32_t wg_reset_stats(wg_ctx *ctx, void *stream);

/* ---- the decode path --------------------------------------------------------------- */

/* Cache probe (paper Section 3.3, global cache keyed by the operator state).
 *   gid, sid  device, B entries
 *   slot      device, B entries: pool row holding the mask of (gid[r], sid[r]), or -1
 * Read-only: nothing is inserted.  1 <= B <= max_batch. */
int32_t wg_mask_cache_lookup(wg_ctx *ctx, const int32_t *gid, const int32_t *sid, int32_t B,
                             int32_t *slot, void *stream);

/* Mask creation (paper Section 1, the third stage of constrained decoding; Section 3.3).
 *   gid, sid          device, B entries
 *   bitmask           device, B rows of W words, row r at bitmask + r * row_stride_words
 *   row_stride_words  >= W
 *   flags             WG_USE_CACHE: rows whose state is cached are copied from the pool; the
 *                     others are built once per distinct state, inserted, then copied.  When
 *                     the pool is full the remaining rows are built straight into `bitmask`.
 *                     WG_NO_CACHE: every row is built, duplicates included.
 * Rows with an unknown grammar or state get an all-zero mask and count as bad_states, on every
 * call that meets them: such a row never takes a cache entry (it also counts as rows_uncached). */
int32_t wg_build_masks(wg_ctx *ctx, const int32_t *gid, const int32_t *sid, int32_t B,
                       uint32_t *bitmask, int64_t row_stride_words, uint32_t flags, void *stream);

/* Mask application (paper Section 1: the mask acts on the logits before a token is sampled),
 * in place.
 *   logits            device, B rows of V elements, row r at logits + r * row_stride_elems;
 *                     1 <= B <= WG_MAX_ROWS
 *   dtype             WG_DTYPE_BF16 or WG_DTYPE_FP32
 *   bitmask           device, as written by wg_build_masks
 *   argmax_out        device, B entries, or NULL.  When given, token[r] = the lowest id among
 *                     the maxima of the allowed logits (-0.0 equals +0.0), or -1 for an
 *                     empty mask.  NaN logits are outside the contract.
 *   workspace         device scratch of wg_apply_workspace_bytes(B) bytes, 8-byte aligned;
 *                     needed only with argmax_out, may be NULL otherwise.  Contents are
 *                     overwritten.
 * Disallowed elements become -inf (bf16 0xFF80, fp32 0xFF800000); all others keep their bits.
 * Fastest when logits is 32-byte aligned and row_stride_elems * element size is a multiple
 * of 32 bytes; other layouts take a slower element-wise kernel with identical results. */
int32_t wg_apply_mask(void *logits, int32_t dtype, int64_t row_stride_elems,
                      const uint32_t *bitmask, int64_t mask_stride_words, int32_t B, int32_t V,
                      int32_t *argmax_out, void *workspace, void *stream);
size_t wg_apply_workspace_bytes(int32_t B);

/* The paper has no counterpart to this call; it exists for deployment reasons only.
 * wg_apply_mask with argmax_out needs a scratch buffer that somebody has to allocate.  Some
 * callers cannot: an inference server that handed every byte of device memory to its own
 * pool at start-up, a plug-in that runs inside someone else's step function where a
 * cudaMalloc would stall the whole device, or a host thread that may not call allocating
 * CUDA routines at all.  For them this variant masks and picks the greedy token exactly as
 * wg_apply_mask does, but keeps its scratch (one 8-byte packed maximum per row) in a fixed
 * array that is part of the library image: WG_NOALLOC_MAX_ROWS * 8 bytes = 32 KB of device
 * memory on every GPU that loads the library, held until the process exits.
 *   arguments   as wg_apply_mask; argmax_out is required (device, B entries)
 *   limit       B <= WG_NOALLOC_MAX_ROWS, otherwise WG_ERR_CAPACITY and nothing is launched
 * The call performs no cudaMalloc, cudaFree or other allocating routine.  The first call on
 * each device looks up the device address of the array (a synchronous query, done with that
 * device current); make that first call outside any stream capture.  Every call on a device
 * uses the same array and begins by clearing the rows it needs, so the previous call's
 * contents never leak in -- but two calls whose kernels can overlap on the GPU (different
 * streams, no ordering between them) race on it and give undefined tokens.  Calls on one
 * stream, or ordered by events, are safe. */
#define WG_NOALLOC_MAX_ROWS 4096
int32_t wg_apply_mask_noalloc(void *logits, int32_t dtype, int64_t row_stride_elems,
                              const uint32_t *bitmask, int64_t mask_stride_words, int32_t B,
                              int32_t V, int32_t *argmax_out, void *stream);

/* State tracking (paper Section 3.2: the current token id updates the state machine).
 *   gid     device, B entries
 *   sid     device, B entries, updated in place
 *   token   device, B entries
 *   status  device, B entries, or NULL: WG_OK, WG_ERR_TOKEN_REJECTED (state unchanged; also
 *           for token ids outside 0..V-1) or WG_ERR_STATE
 *   flags   0 or WG_RESTART_ON_DONE */
int32_t wg_advance(wg_ctx *ctx, const int32_t *gid, int32_t *sid, const int32_t *token,
                   int32_t B, int32_t *status, uint32_t flags, void *stream);

/* One whole decode step on device buffers: cache lookup, build of the misses, mask rows out,
 * apply with greedy argmax, state advance.  Same results as the four calls above in that
 * order, in fewer kernel launches (the rows are copied from the cache pool inside the apply
 * kernel).  Up to 64 rows with 16-byte aligned logits rows the step is ONE launch: every block
 * probes the cache for its row, builds its own part of the mask on a miss, and the last block of
 * a row advances the row's state and files a newly built mask in the cache.  On that path rows
 * that meet the same new state in the same step each build it (masks_built counts every built
 * row, cache_misses every row that missed) and one of them files it.
 * flags: WG_USE_CACHE or WG_NO_CACHE, optionally | WG_RESTART_ON_DONE.
 *   token_out  device, B entries (the greedy choice, -1 for an empty mask), or NULL
 *   status     device, B entries, or NULL (WG_OK, WG_ERR_EMPTY_MASK, WG_ERR_STATE)
 * With token_out NULL the step only masks, for an engine that samples by itself (paper Section 2:
 * the mask is applied to the logits before sampling): lookup, build of the misses, mask rows out
 * and apply run as above, no token is chosen and sid is left as it is; the caller samples from the
 * masked logits and hands its tokens to wg_advance.  status must then be NULL and
 * WG_RESTART_ON_DONE unset (WG_ERR_ARG otherwise). */
int32_t wg_decode_step(wg_ctx *ctx, const int32_t *gid, int32_t *sid, int32_t B, void *logits,
                       int32_t dtype, int64_t row_stride_elems, uint32_t *bitmask,
                       int64_t mask_stride_words, int32_t *token_out, int32_t *status,
                       uint32_t flags, void *stream);

/* The decode step for a vocabulary that is sharded over several GPUs (a tensor-parallel LM
 * head leaves each GPU with logits[:, v_begin:v_end)).  Each GPU runs the step on its own
 * slice -- cache lookup, build of the missing masks for the slice's tokens only, mask words
 * out, apply -- and returns, per row, its best allowed logit and token id packed into one
 * signed 64-bit integer whose signed order is (value, then lower token id first).  The caller
 * takes the maximum over the GPUs (one 8-byte MAX all-reduce per row, e.g. NCCL over NVLink) and
 * hands the result to wg_advance_keys on every GPU, which unpacks the token and advances the
 * states.  The paper has a single mask per request (Section 1); the split follows from rows and
 * tokens being independent and is exact: tokens, states and every masked logit equal those of
 * wg_decode_step on the whole vocabulary.
 *   logits_shard      device, B rows of (v_end - v_begin) elements: element 0 of a row is token
 *                     v_begin; 16-byte aligned rows take the fast kernel
 *   bitmask           device, B rows of W words (the WHOLE vocabulary's width); only the words
 *                     of the slice's tokens are written
 *   v_begin, v_end    0 <= v_begin < v_end <= V; v_begin a multiple of WG_SHARD_ALIGN, v_end a
 *                     multiple of it or V
 *   best_keys         device, B entries, written by this call (smallest value = no allowed token)
 *   flags             WG_USE_CACHE or WG_NO_CACHE
 * With the cache on, a context must always be called with the same slice: cached masks then
 * hold the slice's words only, and calls that would read other words (another slice,
 * wg_decode_step, wg_build_masks with the cache, wg_cache_entry_read) return WG_ERR_ARG until
 * wg_cache_clear.  Masks cached before the first sharded call (wg_cache_prewarm) are complete
 * and stay usable.
 * wg_advance_keys: token_out[r] = the token packed in best_keys[r] (-1: none, status
 * WG_ERR_EMPTY_MASK), then as wg_advance. */
#define WG_SHARD_ALIGN 8192
int32_t wg_decode_step_shard(wg_ctx *ctx, const int32_t *gid, const int32_t *sid, int32_t B,
                             void *logits_shard, int32_t dtype, int64_t row_stride_elems,
                             uint32_t *bitmask, int64_t mask_stride_words, int32_t v_begin,
                             int32_t v_end, int64_t *best_keys, uint32_t flags, void *stream);
int32_t wg_advance_keys(wg_ctx *ctx, const int32_t *gid, int32_t *sid, const int64_t *best_keys,
                        int32_t B, int32_t *token_out, int32_t *status, uint32_t flags,
                        void *stream);

/* A decode step recorded once as a CUDA graph and replayed: where wg_decode_step takes several
 * kernel launches (more than 64 rows) a graph launch replaces them with one call.  (Up to 64
 * rows the step is a single kernel already and a plain call is cheaper than a graph launch.)  All arguments are those of wg_decode_step and
 * are frozen into the graph: the caller keeps writing each step's logits into the same
 * buffer (as an LM head does) and reads tokens and states from the same arrays.  Grammars
 * added to the context after creation are not seen by the graph while the context's grammar
 * registry has not grown (it grows when the 65th, 129th, ... grammar is added); create graphs
 * after the grammars.  wg_step_graph_create records on an internal stream and runs nothing;
 * wg_step_graph_launch enqueues one step on `stream`.  Results are identical to
 * wg_decode_step.  Free the graph before its context. */
typedef struct wg_step_graph wg_step_graph;
int32_t wg_step_graph_create(wg_ctx *ctx, const int32_t *gid, int32_t *sid, int32_t B,
                             void *logits, int32_t dtype, int64_t row_stride_elems,
                             uint32_t *bitmask, int64_t mask_stride_words, int32_t *token_out,
                             int32_t *status, uint32_t flags, wg_step_graph **out);
int32_t wg_step_graph_launch(wg_step_graph *graph, void *stream);
void wg_step_graph_free(wg_step_graph *graph);

/* The same step for a caller whose logits live in HOST memory (pinned memory makes the
 * copies asynchronous): copies logits_host to the device buffer `logits_dev`, runs
 * wg_decode_step, copies the chosen tokens back to token_host and synchronises `stream`.
 *   logits_host  host, B * V elements, rows contiguous
 *   logits_dev   device staging, B rows of row_stride_elems elements
 *   token_dev    device, B entries; token_host host, B entries */
int32_t wg_decode_step_host(wg_ctx *ctx, const int32_t *gid, int32_t *sid, int32_t B,
                            const void *logits_host, void *logits_dev, int32_t dtype,
                            int64_t row_stride_elems, uint32_t *bitmask,
                            int64_t mask_stride_words, int32_t *token_dev, int32_t *token_host,
                            int32_t *status, uint32_t flags, void *stream);

/* ---- diagnostics ------------------------------------------------------------------- */

/* Per-kernel timing for benchmarks.  While enabled, wg_decode_step records CUDA events on the
 * caller's stream around its mask-build kernel and around its apply kernel (at most 8192
 * steps are kept between two reads).  wg_ctx_get_timing waits for the recorded events, adds
 * up the elapsed milliseconds of each kernel over the recorded steps, and forgets them.
 * Any output pointer may be NULL. */
int32_t wg_ctx_set_timing(wg_ctx *ctx, int32_t enable);
int32_t wg_ctx_get_timing(wg_ctx *ctx, double *build_ms, double *apply_ms, int64_t *steps);

/* Work counters of the mask-build kernel, for the benchmark's bound on that kernel (paper
 * Section 1: mask creation is one of the three cost stages; these say what one build costs).
 * While enabled, wg_build_masks / wg_decode_step launch a variant of the build kernel that also
 * counts, over all masks built: the tokens it could not decide 32 at a time and walked through
 * the table, the table look-ups of those walks, and the words of vocabulary masks its word-wise
 * phase read.  The variant is slower; timed runs keep it off.  wg_get_build_work reads the
 * counters (since the last wg_reset_stats) and synchronises `stream`; any pointer may be NULL. */
int32_t wg_ctx_count_build_work(wg_ctx *ctx, int32_t enable);
int32_t wg_get_build_work(wg_ctx *ctx, int64_t *tokens_walked, int64_t *table_lookups,
                          int64_t *mask_words_read, void *stream);

const char *wg_strerror(int32_t status);
/* cudaError_t of the last failed CUDA call on this thread (0 if none). */
int32_t wg_last_cuda_error(void);
/* Number of kernels this library has launched since load (all contexts, all threads). */
int64_t wg_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* WG_H_ */
