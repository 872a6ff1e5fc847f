// Device code of the mask path: build, cache, gather, apply (+ argmax), advance.
// sm_100a; plain integer and load/store work -- nothing here is a dense contraction, so no
// tensor-core instruction appears.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

#include "wg_internal.h"

// ---------------------------------------------------------------------------------------
// device-side views
// ---------------------------------------------------------------------------------------
struct GrammarDev {
    const void *table;          // [n_states][n_classes] of uint16_t (wide == 0) or uint32_t
    const uint8_t *byte_class;  // [256]
    const uint32_t *first_ok;   // [n_states][8] bit b: byte b does not lead to DEAD
    const unsigned long long *leaves;  // [n_states] OR of 1 << (b & 63) over bytes b that
                                       // lead anywhere but back to the state itself
    const int2 *forced;         // [n_states] (token id or -1, next state), or NULL: states of a
                                // token-level Write accept exactly one whole token
    const uint4 *rec_class;     // [V] the vocabulary's 16-byte records with every byte replaced by
                                // its class under THIS grammar's byte_class (shared by grammars
                                // with equal class maps): saves the class look-up in the walk
    const int16_t *leave1;      // [n_states] the byte, if exactly ONE byte leads from the state to a
                                // live state other than itself (a free-text slot's closing byte),
                                // else -1
    const unsigned long long *leave_fold;  // [n_states] for such a state, if it accepts most bytes
                                // and few survive after the leaving byte: the folded set of
                                // bytes that survive in the state after that byte; else 0
    int32_t n_states, n_classes, start, done, eos_class, wide;
};

struct VocabDev {
    const uint4 *rec;         // [V] first 16 bytes of every token, zero padded
    const uint8_t *len;       // [V] min(length, 255)
    const uint32_t *first_mask;  // [256][W] bit t: token t is non-empty and starts with byte b
    const uint32_t *fold_mask;   // [64][W]  bit t: some byte b of token t has (b & 63) == c
    const uint32_t *valid_mask;  // [W]      bit t: token t has at least one byte (EOS has none)
    const uint32_t *offsets;  // [V + 1] CSR, for tokens longer than the record
    const uint8_t *bytes;
    int32_t V, W, eos_id;
};

enum StatSlot {
    ST_HITS = 0, ST_MISSES, ST_BUILT, ST_UNCACHED, ST_REJECTED, ST_EMPTY, ST_BAD_STATE,
    // work counters of the build kernel, only kept by its counting variant (wg_ctx_count_build_work)
    ST_QUEUED,      // tokens that were not decided word-wise and went through the table walk
    ST_WALKED,      // table look-ups of those walks
    ST_MASK_WORDS,  // words of vocabulary masks read by the word-wise phase
    ST_COUNT
};

struct CtxDev {
    const GrammarDev *grammars;
    int32_t n_grammars;
    // mask cache
    unsigned long long *keys;  // [hash_size], 0 = empty, else ((gid + 1) << 32) | sid
    int32_t *vals;             // [hash_size] pool row, or -1 for a key that found the pool full
    uint32_t *pool;            // [capacity][pool_stride]
    int32_t hash_size;         // power of two (0 when capacity == 0)
    int32_t capacity;
    int64_t pool_stride;       // words
    int32_t *n_slots;          // pool rows handed out so far (the high-water mark)
    int32_t *free_rows;        // [capacity] pool rows given back when a grammar was removed
    int32_t *n_free;           // how many of them wait to be handed out again
    // per-call scratch
    int32_t *ent;              // [max_batch] hash entry of each row
    int32_t *slot;             // [max_batch] resolved pool row of each row, or -1
    int32_t *bl_gid, *bl_sid;  // [max_batch] build list
    uint32_t **bl_dst;         // [max_batch] where each listed mask goes
    int32_t *bl_count;
    int32_t *build_next, *build_done;  // work counter of the build kernel and blocks finished;
                                       // both zero between launches
    unsigned long long *argkey;  // [max_batch] packed (value key, ~id) maxima
    unsigned long long *stats;   // [ST_COUNT]
    int32_t *row_done;           // [max_batch] one-launch step: blocks of the row that have finished
                                 // (the last one ends the step for the row); zero between launches
    // "what follows byte b" masks of the vocabulary, made for the bytes that close a free-text
    // slot of some added grammar (see after_masks_kernel); slot k holds AFTER_ROWS rows of W words
    const uint32_t *after_masks; // [AFTER_SLOTS][AFTER_ROWS][W], or NULL while no byte needed them
    const int8_t *after_slot;    // [256] slot of byte b, or -1
    // compact cache (allows / denies storage instead of dense pool rows); pool is NULL then
    int32_t compact;
    uint2 *ent_hdr;                  // [capacity][hdr_stride] per cache row and span of 32 mask
                                     // words: (bitmap of the stored words, where they start in
                                     // the arena | the span's default in bit 31)
    int32_t hdr_stride;              // spans per mask = ceil(W / 32)
    uint32_t *arena;                 // [arena_words] the stored words of all entries
    unsigned long long *arena_top;   // words handed out so far (beyond arena_words: full)
    long long arena_words;           // < 2^31
    int32_t *ent_fail;               // [capacity] 1: part of the entry found no room in the arena;
                                     // the state stays uncached from then on
    int32_t *ent_stage;              // [capacity] staging row that holds the dense mask during
                                     // the call that built the entry
    uint32_t *stage;                 // [max_batch][pool_stride] dense masks built in this call
    int32_t *bl_row;                 // [max_batch] cache row of each build-list entry, or -1
};


constexpr int BUILD_AFTER_MAX_FOLDS = 8;  // larger sets after the leaving byte: no filtering
constexpr int AFTER_SLOTS = 8;   // bytes that can have "what follows" masks
constexpr int AFTER_ROWS = 66;   // row 0: token contains b; row 1: worth a walk whatever follows
                                 // (b is the last byte, or the record ends before the answer is
                                 // known); rows 2 + c: the byte after the first b folds to c
constexpr uint32_t NEG_INF_F32 = 0xFF800000u;
constexpr uint32_t NEG_INF_BF16X2 = 0xFF80FF80u;

__device__ __forceinline__ void pdl_enter();

// ---------------------------------------------------------------------------------------
// table walk
// ---------------------------------------------------------------------------------------
// The token walk (build and advance kernels): state after token t from state s (0 = DEAD).
// The first 16 bytes come as classes straight from the grammar's class-mapped record, so every
// step is one dependent table look-up; longer tokens continue from the CSR bytes.
template <typename T>
__device__ __forceinline__ uint32_t walk_token_classes(const VocabDev &v, const uint4 *rec_class,
                                                       const T *__restrict__ tab, int C,
                                                       const uint8_t *cls, uint32_t s, int t,
                                                       int *lookups = nullptr) {
    // (both loads are issued before the length is looked at: one round trip instead of two;
    // the record of a token without bytes exists and is not used)
    const uint4 rec = __ldg(&rec_class[t]);
    const int n = v.len[t];
    if (n == 0) return 0;
    const uint32_t w[4] = {rec.x, rec.y, rec.z, rec.w};
    // (the index stays in 32 bits: a table has fewer than 2^32 cells, and the address then takes
    // one wide multiply-add instead of a 64-bit multiply, add and shift)
    const uint32_t Cu = (uint32_t)C;
#pragma unroll
    for (int j = 0; j < WG_REC_BYTES; ++j) {
        if (j >= n || s == 0) break;
        s = tab[s * Cu + ((w[j >> 2] >> (8 * (j & 3))) & 0xFFu)];
        if (lookups) ++*lookups;
    }
    if (n > WG_REC_BYTES && s != 0) {
        const uint32_t b = v.offsets[t] + WG_REC_BYTES, e = v.offsets[t + 1];
        for (uint32_t i = b; i < e && s != 0; ++i) {
            s = tab[s * Cu + cls[v.bytes[i]]];
            if (lookups) ++*lookups;
        }
    }
    return s;
}

// ---------------------------------------------------------------------------------------
// Compact cache entries: the adaptive allows / denies storage.  A mask is kept span by span
// (a span = 32 mask words = 1024 tokens).  Each span makes the paper's choice for itself: when
// fewer of its words differ from zero than from all-ones it keeps the allowed side (default
// word 0), otherwise the refused side (default word all-ones below V); only the words that
// differ from the default are stored, back to back in the arena.  The per-span header says
// which words are stored, where they start, and which default applies.  A listed token costs
// at most one stored word, so a mask never takes more room than its id list, and a reader
// finds word w with one header load and one popcount instead of a search.
// ---------------------------------------------------------------------------------------
constexpr uint32_t HDR_DEFAULT_ONES = 0x80000000u;

__device__ __forceinline__ uint32_t full_word(int w, int V, int W) {  // all tokens of word w
    if (w >= W) return 0u;
    const int tail = V & 31;
    return (w == W - 1 && tail) ? ((1u << tail) - 1u) : 0xFFFFFFFFu;
}

// Mask word `span * 32 + lane` of a compact entry (called by all 32 lanes of a warp).
__device__ __forceinline__ uint32_t entry_word(const uint2 *hdr_row, const uint32_t *arena, int span,
                                               int lane, int V, int W) {
    const uint2 hdr = hdr_row[span];
    if ((hdr.x >> lane) & 1u)
        return arena[(hdr.y & ~HDR_DEFAULT_ONES) + __popc(hdr.x & ((1u << lane) - 1u))];
    return (hdr.y & HDR_DEFAULT_ONES) ? full_word(span * 32 + lane, V, W) : 0u;
}

// Stores one finished span (32 mask words, one per lane) of cache row `row`; called by a whole
// warp.  The room is taken with one atomic add that is never given back: the first span that
// does not fit leaves the top beyond the end, and from then on the arena counts as full.
__device__ __forceinline__ void store_span(uint2 *hdr_row, uint32_t *arena,
                                           unsigned long long *arena_top, long long arena_words,
                                           int32_t *fail_flag, unsigned long long *uncached_stat,
                                           int span, uint32_t word, int lane, int V, int W) {
    const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, word != 0u);
    const uint32_t b1 = __ballot_sync(0xFFFFFFFFu, word != full_word(span * 32 + lane, V, W));
    const bool ones = __popc(b1) < __popc(b0);
    uint32_t bits = ones ? b1 : b0;
    const int n = __popc(bits);
    unsigned long long off = 0ull;
    if (n > 0) {
        if (lane == 0) off = atomicAdd(arena_top, (unsigned long long)n);
        off = __shfl_sync(0xFFFFFFFFu, off, 0);
        if (off + (unsigned long long)n > (unsigned long long)arena_words) {
            if (lane == 0 && atomicExch(fail_flag, 1) == 0) atomicAdd(uncached_stat, 1ull);
            bits = 0u;
            off = 0ull;
        } else if ((bits >> lane) & 1u) {
            arena[off + __popc(bits & ((1u << lane) - 1u))] = word;
        }
    }
    if (lane == 0) hdr_row[span] = make_uint2(bits, (uint32_t)off | (ones ? HDR_DEFAULT_ONES : 0u));
}

// ---------------------------------------------------------------------------------------
// What the mask of one (grammar, state) is decided from, and the word-wise decision itself; used
// by the build kernel and by the one-launch step.  The arithmetic is described at the build
// kernel below.
// ---------------------------------------------------------------------------------------
constexpr int BUILD_MAX_FOLDS = 20;    // more leaving folds than this: queue every P token

// The facts about the mask of one (grammar, state), gathered by one warp.
struct MaskFacts {
    const void *table;
    const uint8_t *byte_class;
    const uint4 *rec_class;
    uint32_t *dst;
    const uint32_t *after_rows;     // "what follows the closing byte" masks, or NULL
    unsigned long long leaves, after_fold;
    uint32_t s0, eos_next;
    int32_t gid, n_classes, wide, n_ok, forced_tok, row;
    int32_t n_first, n_fold;        // entries of the two lists below
    uint8_t first_list[128];        // first bytes to OR (or to exclude, when complemented)
    uint8_t fold_list[64];          // folds of the leaving bytes (unused when there are too many)
};

// Called by ONE warp: the grammar record and the state's sets for (gid, sid) into fx.
__device__ __forceinline__ void gather_item_facts(const VocabDev &v, const CtxDev &ctx, int gid_, int sid_,
                                                  uint32_t *dst, int row, bool first_chunk, MaskFacts &fx) {
    const int lane = threadIdx.x & 31;
    uint32_t s_ = (uint32_t)sid_;
    const bool known_ = gid_ >= 0 && gid_ < ctx.n_grammars;
    GrammarDev g = {};
    if (known_) g = ctx.grammars[gid_];
    if (!known_ || s_ >= (uint32_t)g.n_states) s_ = 0;  // unknown state: an all-zero row
    const uint32_t ok_word_ = (s_ && lane < 8) ? g.first_ok[(size_t)s_ * 8 + lane] : 0u;
    int n_ok_ = __popc(ok_word_);
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) n_ok_ += __shfl_xor_sync(0xFFFFFFFFu, n_ok_, o);
    n_ok_ = __shfl_sync(0xFFFFFFFFu, n_ok_, 0);
    const bool complement = n_ok_ > 128;
    // the list of first bytes: byte 32 * j + lane, taken when its bit differs from `complement`
    int n_first_ = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t word = __shfl_sync(0xFFFFFFFFu, ok_word_, j);
        const bool take = (((word >> lane) & 1u) != 0u) != complement;
        const uint32_t m = __ballot_sync(0xFFFFFFFFu, take);
        if (take) fx.first_list[n_first_ + __popc(m & ((1u << lane) - 1u))] = (uint8_t)(32 * j + lane);
        n_first_ += __popc(m);
    }
    const unsigned long long leaves_ = s_ ? g.leaves[s_] : 0ull;
    int n_fold_ = 0;
    if (__popcll(leaves_) <= BUILD_MAX_FOLDS) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const bool take = (leaves_ >> (32 * j + lane)) & 1ull;
            const uint32_t m = __ballot_sync(0xFFFFFFFFu, take);
            if (take) fx.fold_list[n_fold_ + __popc(m & ((1u << lane) - 1u))] = (uint8_t)(32 * j + lane);
            n_fold_ += __popc(m);
        }
    }
    if (lane == 0) {
        fx.gid = known_ ? gid_ : -1;
        fx.s0 = s_;
        fx.dst = dst;
        fx.row = row;
        fx.table = g.table;
        fx.byte_class = g.byte_class;
        fx.rec_class = g.rec_class;
        fx.n_classes = g.n_classes;
        fx.wide = g.wide;
        fx.n_ok = n_ok_;
        fx.n_first = n_first_;
        fx.n_fold = n_fold_;
        fx.leaves = leaves_;
        uint32_t eos_ = 0;
        if (s_) eos_ = g.wide ? static_cast<const uint32_t *>(g.table)[(size_t)s_ * g.n_classes + g.eos_class]
                             : static_cast<const uint16_t *>(g.table)[(size_t)s_ * g.n_classes + g.eos_class];
        fx.eos_next = eos_;
        fx.forced_tok = (s_ && g.forced) ? g.forced[s_].x : -1;  // token-level Write state
        // A free-text slot has ONE byte that leads on (its closing byte); a token that
        // holds it is dead unless that byte ends the token or the byte after its first
        // occurrence survives in the next state.  The vocabulary masks for that byte turn
        // this into word-wise work.
        const uint32_t *rows_ = nullptr;
        unsigned long long fold_ = 0ull;
        if (s_ && ctx.after_masks) {
            const int lv = g.leave1[s_];
            if (lv >= 0) {
                fold_ = g.leave_fold[s_];  // 0: not a state the masks were made for
                const int k_ = fold_ != 0ull ? ctx.after_slot[lv] : -1;
                if (k_ >= 0) rows_ = ctx.after_masks + (size_t)k_ * AFTER_ROWS * v.W;
            }
        }
        fx.after_rows = rows_;
        fx.after_fold = fold_;
        if (first_chunk) {
            atomicAdd(&ctx.stats[ST_BUILT], 1ull);
            if (s_ == 0 && sid_ != 0) atomicAdd(&ctx.stats[ST_BAD_STATE], 1ull);
        }
    }
}

// Mask words w[0..K) of the state described by fx, as far as they can be decided 32 tokens at a
// time: `alive` = tokens allowed without a walk, `todo` = tokens that need the table walk.  A
// negative w[k] is skipped.  The loads of the K words are independent of one another and of every
// branch, so they are all in flight together (one round trip to L2 for the lot).
template <int K, bool COUNT>
__device__ __forceinline__ void decide_words(const VocabDev &v, const MaskFacts &fx, const int (&w)[K],
                                             uint32_t (&alive)[K], uint32_t (&todo)[K],
                                             int &counted_words) {
#pragma unroll
    for (int k = 0; k < K; ++k) { alive[k] = 0; todo[k] = 0; }
    if (fx.forced_tok >= 0) {
#pragma unroll
        for (int k = 0; k < K; ++k)
            if ((fx.forced_tok >> 5) == w[k] && fx.forced_tok < v.V) alive[k] = 1u << (fx.forced_tok & 31);
        return;
    }
    if (fx.s0 == 0) return;
    const int nf = fx.n_first, nq = fx.n_fold;
    const bool complement = fx.n_ok > 128;
    const bool queue_all = __popcll(fx.leaves) > BUILD_MAX_FOLDS;
    uint32_t p[K], q[K];
    size_t at[K];   // a word that is skipped reads word 0 and throws the result away
#pragma unroll
    for (int k = 0; k < K; ++k) { p[k] = 0; q[k] = queue_all ? 0xFFFFFFFFu : 0u; at[k] = w[k] < 0 ? 0 : (size_t)w[k]; }
    for (int i = 0; i < nf; ++i) {
        const uint32_t *row = v.first_mask + (size_t)fx.first_list[i] * v.W;
#pragma unroll
        for (int k = 0; k < K; ++k) p[k] |= __ldg(&row[at[k]]);
    }
    if (complement) {
#pragma unroll
        for (int k = 0; k < K; ++k) p[k] = __ldg(&v.valid_mask[at[k]]) & ~p[k];
    }
    for (int i = 0; i < nq; ++i) {
        const uint32_t *row = v.fold_mask + (size_t)fx.fold_list[i] * v.W;
#pragma unroll
        for (int k = 0; k < K; ++k) q[k] |= __ldg(&row[at[k]]);
    }
    const uint32_t *rows = fx.after_rows;
    uint32_t has[K], worth[K];
#pragma unroll
    for (int k = 0; k < K; ++k) { has[k] = 0; worth[k] = 0; }
    if (rows != nullptr) {   // uniform: loaded whether or not a word turns out to need them
#pragma unroll
        for (int k = 0; k < K; ++k) {
            has[k] = __ldg(&rows[at[k]]);
            worth[k] = __ldg(&rows[(size_t)v.W + at[k]]);
        }
        for (unsigned long long f = fx.after_fold; f; f &= f - 1) {
            const uint32_t *row = rows + (size_t)(2 + __ffsll((long long)f) - 1) * v.W;
#pragma unroll
            for (int k = 0; k < K; ++k) worth[k] |= __ldg(&row[at[k]]);
        }
    }
#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (w[k] < 0) continue;
        uint32_t a = p[k] & ~q[k], t = p[k] & q[k];
        if (rows != nullptr) {
            if (fx.n_ok == 256) {
                // no byte kills the state and only the closing byte leaves it: a token
                // without that byte is allowed without a walk (the folded sets also
                // catch the other bytes of the closing byte's fold, e.g. 'b' for '"')
                a |= t & ~has[k];
                t &= has[k];
            }
            // a token that holds the closing byte is only worth a walk when that byte ends it
            // or the byte after its first occurrence can survive in the next state
            t &= ~has[k] | worth[k];
        }
        if ((v.eos_id >> 5) == w[k] && fx.eos_next != 0) a |= 1u << (v.eos_id & 31);
        alive[k] = a;
        todo[k] = t;
        if (COUNT)
            counted_words += nf + nq + (complement ? 1 : 0) +
                             (rows != nullptr ? 2 + __popcll(fx.after_fold) : 0);
    }
}

// ---------------------------------------------------------------------------------------
// K1: mask build.  Work item = (mask m, chunk of tokens); a fixed-size grid strides over the
// items, so a launch with nothing to build costs a few empty blocks.
//
// Most tokens are decided 32 at a time, without walking the table.  The vocabulary holds
// V-bit masks "token starts with byte b" (256 of them) and "token contains a byte that folds
// to c = b & 63" (64 of them); a state holds the set of first bytes that do not kill it and
// the folded set of bytes that LEAVE it.  For a word of 32 tokens:
//   P = tokens whose first byte keeps the state alive   (OR of a few first-byte masks, or the
//                                                         complement when most bytes are fine)
//   Q = tokens that contain a byte which may leave       (OR of a few fold masks)
//   P & ~Q  are allowed: every byte loops on the state   (free-text states: ~all tokens)
//   ~P      are not allowed                              (literal states: ~all tokens)
//   P & Q   are queued in shared memory and walked afterwards, densely, one per thread.
// ---------------------------------------------------------------------------------------
constexpr int BUILD_THREADS = 256;
constexpr int BUILD_CHUNK_MAX = 8192;  // tokens per work item (the launch picks 2048 or 8192)

// The spans of one finished chunk (n_words mask words in shared memory, beginning at span
// first_span) into a cache row.
__device__ __forceinline__ void store_chunk_spans(uint2 *hdr_row, uint32_t *arena,
                                               unsigned long long *arena_top, long long arena_words,
                                               int32_t *fail_flag, unsigned long long *uncached_stat,
                                               int first_span, int n_words, const uint32_t *words,
                                               int V, int W) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int sl = warp; sl * 32 < n_words; sl += (int)(blockDim.x >> 5)) {
        const int wl = sl * 32 + lane;
        store_span(hdr_row, arena, arena_top, arena_words, fail_flag, uncached_stat, first_span + sl,
                   wl < n_words ? words[wl] : 0u, lane, V, W);
    }
}

struct BuildWork {
    const int32_t *gid, *sid;   // per entry
    uint32_t *const *dst_list;  // per entry destination, or NULL: use dst_base + m * dst_stride
    uint32_t *dst_base;
    int64_t dst_stride;
    const int32_t *count_ptr;   // number of entries on the device, or NULL: use count
    int32_t count;
    int32_t chunk;              // tokens per work item: a multiple of 32, <= BUILD_CHUNK_MAX
    int32_t t_first, t_last;    // tokens [t_first, t_last) are built: whole chunks, or up to W * 32
};

// COMPACT: the cache keeps allows / denies entries; finished chunks are also stored as spans.
// COUNT: the variant that also counts its work (queued tokens, table look-ups, vocabulary-mask
// words read) for the benchmark's bound; never used for a timed launch.
template <bool COMPACT, bool COUNT = false>
__global__ void __launch_bounds__(BUILD_THREADS, (COMPACT || COUNT) ? 5 : 8)
build_masks_kernel(VocabDev v, CtxDev ctx, BuildWork work) {
    // the facts about one work item's mask, gathered by warp 0 (two copies: the next item's are
    // gathered while the other warps walk the current item's tokens)
    __shared__ MaskFacts facts[2];
    __shared__ uint32_t words[BUILD_CHUNK_MAX / 32];
    __shared__ uint16_t todo[BUILD_CHUNK_MAX];
    __shared__ int n_todo;
    __shared__ uint32_t next_item;
    pdl_enter();
    const int lane = threadIdx.x & 31;
    const int n_entries = work.count_ptr ? *work.count_ptr : work.count;
    const int n_chunks = (work.t_last - work.t_first + work.chunk - 1) / work.chunk;
    // (item numbers stay in 32 bits: the launch refuses more than 2^31 of them; the division by
    // the chunk count below would otherwise be a 64-bit one, a hundred instructions per item)
    const uint32_t n_items = (uint32_t)n_entries * (uint32_t)n_chunks;
    // Nothing to build (every row of a warm step hit the cache): leave at once.  Nobody has
    // touched the work counters, so they need no reset either -- and the launch is then a few
    // hundred blocks that read one word and exit, on the critical path of every warm step.
    if (n_items == 0) return;

    // Called by warp 0: the facts of item `it` into fx.
    auto gather = [&](uint32_t it, MaskFacts &fx) {
        const int m = (int)(it / (uint32_t)n_chunks);
        const int chunk = (int)(it - (uint32_t)m * (uint32_t)n_chunks);
        uint32_t *dst = work.dst_list ? work.dst_list[m] : work.dst_base + (int64_t)m * work.dst_stride;
        const int row = (COMPACT && work.dst_list) ? ctx.bl_row[m] : -1;
        gather_item_facts(v, ctx, work.gid[m], work.sid[m], dst, row, chunk == 0, fx);
    };

    if (threadIdx.x == 0) n_todo = 0;
    if (threadIdx.x < 32 && blockIdx.x < n_items) gather(blockIdx.x, facts[0]);
    __syncthreads();
    // Items differ a lot in cost (a literal state decides nearly everything word-wise, a
    // free-text state walks thousands of tokens), so after its first item a block takes the next
    // one from a device counter instead of a fixed stride.  Warp 0 does that, and gathers the
    // next item's facts, while the other seven warps walk the current item's queued tokens.
    int cur = 0;
    for (uint32_t item = blockIdx.x; item < n_items; item = next_item, cur ^= 1) {
        const MaskFacts &info = facts[cur];
        const int m = (int)(item / (uint32_t)n_chunks);
        const int t_begin = work.t_first + (int)(item - (uint32_t)m * (uint32_t)n_chunks) * work.chunk;
        const int t_end = min(t_begin + work.chunk, work.t_last);
        // phase 1: one word of 32 tokens per thread
        const int n_words = (t_end - t_begin) >> 5;
        int counted_words = 0, counted_lookups = 0;
        for (int wl = threadIdx.x; wl < ((n_words + 31) & ~31); wl += BUILD_THREADS) {
            const int w[1] = {wl < n_words ? (t_begin >> 5) + wl : -1};
            uint32_t alive[1], queue[1];
            decide_words<1, COUNT>(v, info, w, alive, queue, counted_words);
            if (wl < n_words) words[wl] = alive[0];
            // queue the undecided tokens: one shared-memory atomic per warp
            const int mine = __popc(queue[0]);
            int before = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int x = __shfl_up_sync(0xFFFFFFFFu, before, o);
                if (lane >= o) before += x;
            }
            int base = 0;
            if (lane == 31 && before > 0) base = atomicAdd(&n_todo, before);
            base = __shfl_sync(0xFFFFFFFFu, base, 31) + before - mine;
            uint32_t bits = queue[0];
            while (bits) {
                const int bit = __ffs(bits) - 1;
                bits &= bits - 1;
                todo[base++] = (uint16_t)(wl * 32 + bit);
            }
        }
        __syncthreads();
        // phase 2: warp 0 takes the block's next item and gathers its facts; the other warps
        // walk the queued tokens, one per thread (the EOS token is never queued: it has no bytes)
        const int n = n_todo;
        if (threadIdx.x < 32) {
            uint32_t nxt = 0;
            if (lane == 0) nxt = gridDim.x + (uint32_t)atomicAdd(ctx.build_next, 1);
            nxt = __shfl_sync(0xFFFFFFFFu, nxt, 0);
            if (lane == 0) next_item = nxt;
            if (nxt < n_items) gather(nxt, facts[cur ^ 1]);
        } else {
            for (int i = threadIdx.x - 32; i < n; i += BUILD_THREADS - 32) {
                const int rel = todo[i];
                int *const counter = COUNT ? &counted_lookups : nullptr;
                const uint32_t end = info.wide
                    ? walk_token_classes<uint32_t>(v, info.rec_class, static_cast<const uint32_t *>(info.table),
                                                   info.n_classes, info.byte_class, info.s0, t_begin + rel, counter)
                    : walk_token_classes<uint16_t>(v, info.rec_class, static_cast<const uint16_t *>(info.table),
                                                   info.n_classes, info.byte_class, info.s0, t_begin + rel, counter);
                if (end != 0) atomicOr(&words[rel >> 5], 1u << (rel & 31));
            }
        }
        if (COUNT) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                counted_words += __shfl_xor_sync(0xFFFFFFFFu, counted_words, o);
                counted_lookups += __shfl_xor_sync(0xFFFFFFFFu, counted_lookups, o);
            }
            if (lane == 0) {
                atomicAdd(&ctx.stats[ST_MASK_WORDS], (unsigned long long)counted_words);
                atomicAdd(&ctx.stats[ST_WALKED], (unsigned long long)counted_lookups);
            }
            if (threadIdx.x == 32) atomicAdd(&ctx.stats[ST_QUEUED], (unsigned long long)n);
        }
        __syncthreads();
        if (threadIdx.x == 0) n_todo = 0;  // everybody has read it
        // phase 3: whole words out
        uint32_t *dst = info.dst;
        for (int wl = threadIdx.x; wl < n_words; wl += BUILD_THREADS)
            dst[(t_begin >> 5) + wl] = words[wl];
        // Compact cache: the chunk's spans go into the cache entry straight from shared memory
        // (chunks are whole spans; the dense words above only serve the call that built them).
        if (COMPACT && info.row >= 0)
            store_chunk_spans(ctx.ent_hdr + (int64_t)info.row * ctx.hdr_stride, ctx.arena, ctx.arena_top,
                              ctx.arena_words, ctx.ent_fail + info.row, ctx.stats + ST_UNCACHED,
                              t_begin >> 10, n_words, words, v.V, v.W);
        __syncthreads();  // the shared arrays are free for the next item
    }
    // the last block to leave puts the counters back to zero for the next launch
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(ctx.build_done, 1) == (int)gridDim.x - 1) {
            *ctx.build_next = 0;
            *ctx.build_done = 0;
        }
    }
}

// ---------------------------------------------------------------------------------------
// Warp-level queue of undecided tokens for a mask build inside another kernel (the one-launch
// step): a warp decides whole spans 32 tokens per lane at a time, queues the undecided tokens in
// its own slice of shared memory, walks them and ends with the spans' finished words in registers,
// one word per lane -- the layout the apply sweeps take their mask words in.
// ---------------------------------------------------------------------------------------
constexpr int WARP_QUEUE = 1024;   // queued tokens per warp: one whole span always fits

// Walks the tokens a warp has queued (entries: span slot k << 10 | token within the span) and
// ORs the survivors into the warp's scratch words; called by the whole warp.
template <bool COUNT>
__device__ __forceinline__ void walk_queued(const VocabDev &v, const MaskFacts &fx, const uint16_t *queue,
                                            int n, int t_base, int span_step, uint32_t *scratch,
                                            int &counted_lookups) {
    const int lane = threadIdx.x & 31;
    __syncwarp();
    for (int i = lane; i < n; i += 32) {
        const int e = queue[i];
        const int k = e >> 10, rel = e & 1023;
        const int t = t_base + k * span_step + rel;
        int *const counter = COUNT ? &counted_lookups : nullptr;
        const uint32_t end = fx.wide
            ? walk_token_classes<uint32_t>(v, fx.rec_class, static_cast<const uint32_t *>(fx.table),
                                           fx.n_classes, fx.byte_class, fx.s0, t, counter)
            : walk_token_classes<uint16_t>(v, fx.rec_class, static_cast<const uint16_t *>(fx.table),
                                           fx.n_classes, fx.byte_class, fx.s0, t, counter);
        if (end != 0) atomicOr(&scratch[k * 32 + (rel >> 5)], 1u << (rel & 31));
    }
    __syncwarp();
}

// Appends the set bits of todo[k], for the span slots k named in `slots`, to the warp's queue
// (which holds `queued` entries); returns the new count.  Called by the whole warp.
template <int K>
__device__ __forceinline__ int push_queued(uint16_t *queue, int queued, const uint32_t (&todo)[K],
                                           uint32_t slots) {
    const int lane = threadIdx.x & 31;
    int n_mine = 0;
#pragma unroll
    for (int k = 0; k < K; ++k)
        if ((slots >> k) & 1u) n_mine += __popc(todo[k]);
    int before = n_mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int x = __shfl_up_sync(0xFFFFFFFFu, before, o);
        if (lane >= o) before += x;
    }
    const int total = __shfl_sync(0xFFFFFFFFu, before, 31);
    int at = queued + before - n_mine;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (!((slots >> k) & 1u)) continue;
        uint32_t bits = todo[k];
        while (bits) {
            const int bit = __ffs(bits) - 1;
            bits &= bits - 1;
            queue[at++] = (uint16_t)((k << 10) | (lane * 32 + bit));
        }
    }
    return queued + total;
}

// ---------------------------------------------------------------------------------------
// Set-up kernels of wg_ctx_add_grammar (a grammar that is instantiated per request is added on
// the request's critical path, so its derived arrays are made here rather than on the host).
// ---------------------------------------------------------------------------------------

// Per state: first_ok (256 bits: bytes that do not lead to DEAD) and leaves (64 bits: folds
// b & 63 of the bytes that lead anywhere but back to the state).  One block of 256 threads per
// state, thread b looks at byte b; state 0 (DEAD) gets zeros.
template <typename T>
__global__ void __launch_bounds__(256)
grammar_state_info_kernel(const T *__restrict__ table, const uint8_t *__restrict__ byte_class,
                          int n_states, int n_classes, uint32_t *first_ok,
                          unsigned long long *leaves, int16_t *leave1) {
    __shared__ uint32_t out_bits[8];
    const int st = blockIdx.x;
    if (st >= n_states) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t to = st == 0 ? 0u : (uint32_t)table[(size_t)st * n_classes + byte_class[threadIdx.x]];
    const uint32_t ok = __ballot_sync(0xFFFFFFFFu, to != 0u);
    const uint32_t out = __ballot_sync(0xFFFFFFFFu, st != 0 && to != (uint32_t)st);
    if (lane == 0) {
        first_ok[(size_t)st * 8 + warp] = ok;
        out_bits[warp] = out;
    }
    __syncthreads();
    if (threadIdx.x == 0) {  // byte b = 32 * warp + lane folds to 32 * (warp & 1) + lane
        const uint32_t lo = out_bits[0] | out_bits[2] | out_bits[4] | out_bits[6];
        const uint32_t hi = out_bits[1] | out_bits[3] | out_bits[5] | out_bits[7];
        leaves[st] = ((unsigned long long)hi << 32) | lo;
    }
    // bytes that lead to a LIVE state other than the state itself: exactly one?
    const uint32_t away = __ballot_sync(0xFFFFFFFFu, st != 0 && to != 0u && to != (uint32_t)st);
    __syncthreads();
    if (lane == 0) out_bits[warp] = away;
    __syncthreads();
    if (threadIdx.x == 0) {
        int n = 0, byte = -1;
        for (int w = 0; w < 8; ++w) {
            n += __popc(out_bits[w]);
            if (out_bits[w]) byte = w * 32 + __ffs(out_bits[w]) - 1;
        }
        leave1[st] = (int16_t)(n == 1 ? byte : -1);
    }
}

// Second pass, one thread per state: for a state with a single leaving byte, the folded set of
// bytes that survive right after it; and one bit per byte value that is such a leaving byte with
// a small set after it (bits: 8 words, zeroed before) -- those bytes get "what follows" masks.
template <typename T>
__global__ void leave_info_kernel(const T *__restrict__ table, const uint8_t *__restrict__ byte_class,
                                  const uint32_t *__restrict__ first_ok, const int16_t *leave1,
                                  int n_states, int n_classes, unsigned long long *leave_fold,
                                  uint32_t *bits) {
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= n_states) return;
    const int b = leave1[s];
    unsigned long long fold = 0ull;
    if (b >= 0) {
        const uint32_t s1 = (uint32_t)table[(size_t)s * n_classes + byte_class[b]];
        const uint32_t *ok1 = first_ok + (size_t)s1 * 8;
        fold = (unsigned long long)(ok1[0] | ok1[2] | ok1[4] | ok1[6]) |
               ((unsigned long long)(ok1[1] | ok1[3] | ok1[5] | ok1[7]) << 32);
        // masks are only worth making for states that accept most bytes (free-text slots): a
        // state inside a literal queues few tokens anyway
        int n_ok = 0;
        for (int i = 0; i < 8; ++i) n_ok += __popc(first_ok[(size_t)s * 8 + i]);
        if (n_ok > 128 && __popcll(fold) <= BUILD_AFTER_MAX_FOLDS) atomicOr(&bits[b >> 5], 1u << (b & 31));
        else fold = 0ull;
    }
    leave_fold[s] = fold;
}

// The "what follows byte b" masks of one byte (AFTER_ROWS rows of W words, zeroed before).
// One thread per token, a warp per mask word.  Only the first 16 bytes of a token are looked at;
// where they do not settle the question the token is marked as worth a walk.
__global__ void after_masks_kernel(VocabDev v, int b, uint32_t *rows) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;  // grid covers W * 32 tokens
    const int w = t >> 5;
    if (w >= v.W) return;
    int fold = -1;            // fold of the byte after the first b, if the record shows it
    bool has = false, always = false;
    if (t < v.V) {
        const int n = v.len[t];
        const uint4 r = v.rec[t];
        const uint32_t word[4] = {r.x, r.y, r.z, r.w};
        const int seen = n < WG_REC_BYTES ? n : WG_REC_BYTES;
        int pos = -1;
        for (int j = seen - 1; j >= 0; --j)
            if (((word[j >> 2] >> (8 * (j & 3))) & 0xFFu) == (uint32_t)b) pos = j;
        if (pos >= 0) {
            has = true;
            if (pos + 1 < seen) fold = (int)((word[(pos + 1) >> 2] >> (8 * ((pos + 1) & 3))) & 63u);
            else always = true;  // b ends the token, or what follows lies beyond the record
        } else if (n > WG_REC_BYTES) {
            has = true;          // b may occur further on
            always = true;
        }
    }
    const uint32_t m_has = __ballot_sync(0xFFFFFFFFu, has);
    const uint32_t m_always = __ballot_sync(0xFFFFFFFFu, always);
    const uint32_t peers = __match_any_sync(0xFFFFFFFFu, fold);
    const int lane = threadIdx.x & 31;
    if (lane == 0) {
        rows[w] = m_has;
        rows[(size_t)v.W + w] = m_always;
    }
    if (fold >= 0 && lane == __ffs(peers) - 1) rows[(size_t)(2 + fold) * v.W + w] = peers;
}

// The vocabulary's 16-byte records with every byte replaced by its class.
__global__ void map_records_kernel(const uint4 *__restrict__ rec, const uint8_t *__restrict__ byte_class,
                                   uint4 *out, int V) {
    __shared__ uint8_t cls[256];
    for (int i = threadIdx.x; i < 256; i += blockDim.x) cls[i] = byte_class[i];
    __syncthreads();
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= V) return;
    const uint4 r = rec[t];
    uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
        w[i] = (uint32_t)cls[w[i] & 0xFFu] | ((uint32_t)cls[(w[i] >> 8) & 0xFFu] << 8) |
               ((uint32_t)cls[(w[i] >> 16) & 0xFFu] << 16) | ((uint32_t)cls[w[i] >> 24] << 24);
    out[t] = make_uint4(w[0], w[1], w[2], w[3]);
}

// ---------------------------------------------------------------------------------------
// K2: mask cache.  Open addressing with linear probing over 64-bit keys.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long cache_key(int gid, int sid) {
    return ((unsigned long long)(uint32_t)(gid + 1) << 32) | (uint32_t)sid;
}

__device__ __forceinline__ uint32_t cache_hash(unsigned long long k) {
    k ^= k >> 33; k *= 0xFF51AFD7ED558CCDull; k ^= k >> 33; k *= 0xC4CEB9FE1A85EC53ull; k ^= k >> 33;
    return (uint32_t)k;
}

constexpr int32_t ENT_NEW = 0x40000000;  // marks the row that inserted its key in this call
// The key of an entry whose grammar was removed: it matches no state and does not end a probe
// sequence (grammar ids stay below 65 535, so no real key has all bits set).
constexpr unsigned long long KEY_REMOVED = ~0ull;

// No pool row left to hand out (neither a returned one nor a fresh one).
__device__ __forceinline__ bool pool_full(const CtxDev &ctx) {
    return *(volatile int32_t *)ctx.n_slots >= ctx.capacity && *(volatile int32_t *)ctx.n_free <= 0;
}

// A pool row for a new entry: one that a removed grammar gave back, else a fresh one; -1 when
// the pool is full.  (Rows are only given back by remove_grammar_entries_kernel, which never
// runs beside a kernel that takes rows.)
__device__ __forceinline__ int32_t take_pool_row(const CtxDev &ctx) {
    const int32_t waiting = atomicSub(ctx.n_free, 1);
    if (waiting > 0) return ctx.free_rows[waiting - 1];
    atomicAdd(ctx.n_free, 1);
    const int32_t row = atomicAdd(ctx.n_slots, 1);
    if (row < ctx.capacity) return row;
    atomicSub(ctx.n_slots, 1);
    return -1;
}

// Read-only probe for (g, s): the pool row; -1 when the key is absent; -2 when it is present
// without a usable row (taken while the pool was full, being filed at this moment, or a compact
// entry that found no room in the arena).
__device__ __forceinline__ int32_t cache_probe(const CtxDev &ctx, int g, int s) {
    if (ctx.hash_size <= 0) return -1;
    const unsigned long long key = cache_key(g, s);
    const uint32_t mask = (uint32_t)ctx.hash_size - 1;
    uint32_t h = cache_hash(key) & mask;
    for (int probe = 0; probe < ctx.hash_size; ++probe, h = (h + 1) & mask) {
        const unsigned long long k = ctx.keys[h];
        if (k == key) {
            const int32_t row = *(volatile int32_t *)&ctx.vals[h];
            if (row < 0 || (ctx.compact && ctx.ent_fail[row])) return -2;
            return row;
        }
        if (k == 0) break;
    }
    return -1;
}

// Read-only probe: slot[r] = pool row or -1.
__global__ void cache_lookup_kernel(CtxDev ctx, const int32_t *gid, const int32_t *sid, int B,
                                    int32_t *slot) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= B) return;
    int32_t found = -1;
    if (ctx.hash_size > 0) {
        const unsigned long long key = cache_key(gid[r], sid[r]);
        const uint32_t mask = (uint32_t)ctx.hash_size - 1;
        uint32_t h = cache_hash(key) & mask;
        for (int probe = 0; probe < ctx.hash_size; ++probe, h = (h + 1) & mask) {
            const unsigned long long k = ctx.keys[h];
            if (k == key) { found = ctx.vals[h]; break; }
            if (k == 0) break;
        }
        if (ctx.compact && found >= 0 && ctx.ent_fail[found]) found = -1;
    }
    slot[r] = found;
}

// Lookup-or-insert for one batch, run by ONE block so that a block barrier separates "every
// key of the batch is in the table and owns a pool row" from "read the rows back".  Rows whose
// state is new append one build-list entry per distinct state; when the pool or the table is
// full the row is listed for an uncached build straight into its bitmask row.
// bitmask may be NULL (prewarm): uncached rows are then dropped.
//
// The kernel sits between the previous step's advance and this step's apply with nothing to hide
// its latency, so the usual case -- the state is cached and found at its first probe position --
// is kept to two round trips after the wait: the state id, then key and pool row together.  What
// never changes while steps are in flight (the row's grammar id, that grammar's state count) is
// read before the wait, for the first row of every thread.
__global__ void __launch_bounds__(1024)
cache_lookup_insert_kernel(CtxDev ctx, const int32_t *gid, const int32_t *sid, int B,
                           uint32_t *bitmask, int64_t mask_stride) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int g_first = (int)threadIdx.x < B ? gid[threadIdx.x] : -1;
    const int n_first = (g_first >= 0 && g_first < ctx.n_grammars) ? ctx.grammars[g_first].n_states : 0;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (threadIdx.x == 0) *ctx.bl_count = 0;
    __syncthreads();
    const uint32_t mask = (uint32_t)ctx.hash_size - 1;
    int hits = 0, misses = 0, uncached = 0;
    unsigned long long settled = 0ull;  // bit i: the i-th row of this thread was served below
    int it = 0;
    for (int r = threadIdx.x; r < B; r += blockDim.x, ++it) {
        ctx.argkey[r] = 0ull;
        const int s = sid[r];
        const int g = it == 0 ? g_first : gid[r];
        const int n_states = it == 0 ? n_first : ((g >= 0 && g < ctx.n_grammars) ? ctx.grammars[g].n_states : 0);
        int32_t entry = -1;
        bool inserted = false;
        // a state id that the grammar does not have (or DEAD) gets no cache entry: the row is
        // built uncached, as a row of zeros, and counted as a bad state on every step
        if (ctx.hash_size > 0 && s > 0 && s < n_states) {
            const unsigned long long key = cache_key(g, s);
            uint32_t h = cache_hash(key) & mask;
            {
                // key and pool row of the first probe position, requested together.  A row >= 0
                // under the right key is final: rows are written once, after the key.
                const unsigned long long k0 = ctx.keys[h];
                const int32_t row0 = *(volatile int32_t *)&ctx.vals[h];
                if (k0 == key && row0 >= 0 && !(ctx.compact && ctx.ent_fail[row0]) && it < 64) {
                    ctx.slot[r] = row0;
                    ++hits;
                    settled |= 1ull << it;
                    continue;
                }
            }
            for (int probe = 0; probe < ctx.hash_size; ++probe, h = (h + 1) & mask) {
                unsigned long long k = ctx.keys[h];
                if (k == 0) {
                    // a full pool takes no new keys, so the table never fills up with states
                    // it cannot serve (the row is then built uncached)
                    if (pool_full(ctx)) break;
                    k = atomicCAS(&ctx.keys[h], 0ull, key);
                    if (k == 0) {  // this thread owns the new entry
                        const int32_t row = take_pool_row(ctx);
                        if (row >= 0) {
                            ctx.vals[h] = row;
                            const int i = atomicAdd(ctx.bl_count, 1);
                            ctx.bl_gid[i] = g;
                            ctx.bl_sid[i] = s;
                            if (ctx.compact) {  // built into a staging row; its spans also go to the arena
                                ctx.bl_dst[i] = ctx.stage + (int64_t)i * ctx.pool_stride;
                                ctx.bl_row[i] = row;
                                ctx.ent_fail[row] = 0;
                                ctx.ent_stage[row] = i;
                            } else {
                                ctx.bl_dst[i] = ctx.pool + (int64_t)row * ctx.pool_stride;
                            }
                        } else {
                            ctx.vals[h] = -1;
                        }
                        entry = (int32_t)h;
                        inserted = true;
                        break;
                    }
                }
                if (k == key) { entry = (int32_t)h; break; }
            }
        }
        ctx.ent[r] = (entry >= 0 && inserted) ? (entry | ENT_NEW) : entry;
    }
    __syncthreads();
    it = 0;
    for (int r = threadIdx.x; r < B; r += blockDim.x, ++it) {
        if (it < 64 && ((settled >> it) & 1ull)) continue;
        const int32_t e = ctx.ent[r];
        int32_t row = e >= 0 ? ctx.vals[e & ~ENT_NEW] : -1;
        // a state whose entry found no room in the arena is rebuilt on every step (a row
        // inserted by this very call still has the flag clear here)
        if (ctx.compact && row >= 0 && ctx.ent_fail[row]) row = -1;
        ctx.slot[r] = row;
        // a hit is a row served from a pool row that some earlier row or call already owned
        if (row >= 0 && !(e & ENT_NEW)) ++hits; else ++misses;
        if (row < 0) {
            ++uncached;
            if (bitmask) {
                const int i = atomicAdd(ctx.bl_count, 1);
                ctx.bl_gid[i] = gid[r];
                ctx.bl_sid[i] = sid[r];
                ctx.bl_dst[i] = bitmask + (int64_t)r * mask_stride;
                if (ctx.compact) ctx.bl_row[i] = -1;
            }
        }
    }
    // one atomic per warp and counter instead of one per row
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        hits += __shfl_xor_sync(0xFFFFFFFFu, hits, o);
        misses += __shfl_xor_sync(0xFFFFFFFFu, misses, o);
        uncached += __shfl_xor_sync(0xFFFFFFFFu, uncached, o);
    }
    if ((threadIdx.x & 31) == 0) {
        if (hits) atomicAdd(&ctx.stats[ST_HITS], (unsigned long long)hits);
        if (misses) atomicAdd(&ctx.stats[ST_MISSES], (unsigned long long)misses);
        if (uncached) atomicAdd(&ctx.stats[ST_UNCACHED], (unsigned long long)uncached);
    }
}

// Rows of a WG_NO_CACHE step: no pool row, and the packed maxima start at zero.
__global__ void reset_rows_kernel(CtxDev ctx, int B) {
    pdl_enter();
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < B) { ctx.slot[r] = -1; ctx.argkey[r] = 0ull; }
}

__global__ void cache_clear_kernel(CtxDev ctx) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < ctx.hash_size) { ctx.keys[i] = 0ull; ctx.vals[i] = -1; }
    if (i == 0) {
        *ctx.n_slots = 0;
        *ctx.n_free = 0;
        if (ctx.compact) *ctx.arena_top = 0ull;
    }
}

// wg_ctx_remove_grammar: every cache entry of grammar g stops matching (its key becomes
// KEY_REMOVED, so probe sequences that pass over it stay whole) and its pool row goes onto the list
// of rows to hand out again.  counts[0] += entries dropped.  Runs alone on an idle device.
__global__ void remove_grammar_entries_kernel(CtxDev ctx, int g, int32_t *counts) {
    const int h = blockIdx.x * blockDim.x + threadIdx.x;
    if (h >= ctx.hash_size) return;
    if ((uint32_t)(ctx.keys[h] >> 32) != (uint32_t)(g + 1)) return;
    const int32_t row = ctx.vals[h];
    ctx.keys[h] = KEY_REMOVED;
    ctx.vals[h] = -1;
    if (row >= 0) ctx.free_rows[atomicAdd(ctx.n_free, 1)] = row;
    atomicAdd(&counts[0], 1);
}

// Rebuilds the hash table from a copy of itself without the removed entries (they would
// otherwise lengthen every probe sequence for good).  old_keys / old_vals: the copy; the
// table itself has been cleared before.
__global__ void rehash_kernel(CtxDev ctx, const unsigned long long *old_keys, const int32_t *old_vals) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= ctx.hash_size) return;
    const unsigned long long key = old_keys[i];
    if (key == 0ull || key == KEY_REMOVED) return;
    const uint32_t mask = (uint32_t)ctx.hash_size - 1;
    uint32_t h = cache_hash(key) & mask;
    for (int probe = 0; probe < ctx.hash_size; ++probe, h = (h + 1) & mask) {
        if (atomicCAS(&ctx.keys[h], 0ull, key) == 0ull) {
            ctx.vals[h] = old_vals[i];
            return;
        }
    }
}

__global__ void iota_states_kernel(int32_t *gid, int32_t *sid, int g, int first, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) { gid[i] = g; sid[i] = first + i; }
}

// K3 for the compact cache: expand entries into bitmask rows.  grid = (chunks of 32 spans, B).
__global__ void __launch_bounds__(256)
cache_gather_compact_kernel(CtxDev ctx, int V, int W, uint32_t *bitmask, int64_t mask_stride) {
    const int r = blockIdx.y;
    const int32_t row = ctx.slot[r];
    if (row < 0) return;  // built straight into the bitmask
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_spans = (W + 31) / 32;
    const bool failed = ctx.ent_fail[row] != 0;
    const uint2 *hdr_row = ctx.ent_hdr + (int64_t)row * ctx.hdr_stride;
    uint32_t *dst = bitmask + (int64_t)r * mask_stride;
    for (int span = blockIdx.x * 32 + warp; span < min(n_spans, (int)(blockIdx.x + 1) * 32); span += 8) {
        const int w = span * 32 + lane;
        uint32_t word;
        if (!failed)
            word = entry_word(hdr_row, ctx.arena, span, lane, V, W);
        else  // built in this call and the arena had no room: the staging row still holds it
            word = w < W ? ctx.stage[(int64_t)ctx.ent_stage[row] * ctx.pool_stride + w] : 0u;
        if (w < W) dst[w] = word;
    }
}

// K3: copy cached rows out.  grid = (chunks, B).
__global__ void cache_gather_kernel(CtxDev ctx, int W, uint32_t *bitmask, int64_t mask_stride) {
    const int r = blockIdx.y;
    const int32_t row = ctx.slot[r];
    if (row < 0) return;  // built straight into the bitmask
    const uint32_t *src = ctx.pool + (int64_t)row * ctx.pool_stride;
    uint32_t *dst = bitmask + (int64_t)r * mask_stride;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < W; i += gridDim.x * blockDim.x)
        dst[i] = src[i];
}

// ---------------------------------------------------------------------------------------
// K4 / K5: apply (+ greedy argmax).
//
// Fast kernel: a warp covers 2 KB of one logits row per pass with four 512-byte fully
// coalesced 16-byte-per-lane accesses; lane l first loads mask word l of the span (one
// coalesced 128-byte load), and each lane then fetches "its" word for every access by
// shuffle.  Per 16-byte chunk: all bits clear -> store -inf without loading; all bits set ->
// touch nothing (load only for the argmax); mixed -> load, patch, store.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t order_key(uint32_t f32_bits) {
    if (f32_bits == 0x80000000u) f32_bits = 0;  // -0.0 ties with +0.0
    return (f32_bits & 0x80000000u) ? ~f32_bits : (f32_bits | 0x80000000u);
}

__device__ __forceinline__ unsigned long long pack_best(uint32_t key, int idx) {
    return ((unsigned long long)key << 32) | (uint32_t)(0xFFFFFFFFu - (uint32_t)idx);
}

__device__ __forceinline__ int unpack_best(unsigned long long k) {
    return k == 0ull ? -1 : (int)(0xFFFFFFFFu - (uint32_t)(k & 0xFFFFFFFFull));
}

template <typename E> struct ElemTraits;
template <> struct ElemTraits<uint16_t> {  // bf16
    static constexpr int PER_CHUNK = 8;    // elements per 16-byte chunk
    static __device__ __forceinline__ uint32_t f32_bits(uint16_t e) { return (uint32_t)e << 16; }
    static constexpr uint32_t NEG_INF = 0xFF80u;
};
template <> struct ElemTraits<uint32_t> {  // fp32
    static constexpr int PER_CHUNK = 4;
    static __device__ __forceinline__ uint32_t f32_bits(uint32_t e) { return e; }
    static constexpr uint32_t NEG_INF = 0xFF800000u;
};

constexpr int APPLY_THREADS = 256;
constexpr int APPLY_WARPS = APPLY_THREADS / 32;
constexpr int APPLY_SPANS_PER_WARP = 4;  // a block covers at most 8 * 4 spans = 32768 tokens

struct ApplyArgs {
    void *logits;
    int64_t row_stride;       // elements
    const uint32_t *bitmask;  // row source when the row has no pool slot
    uint32_t *bitmask_out;    // GATHER: where pool rows are copied to (same array as bitmask)
    int64_t mask_stride;      // words
    int32_t B, V, W;
    int32_t spans_per_block;  // spans (32 mask words) each block handles
    int32_t span_first;       // vocabulary shard: the first span that is handled.  `logits` then
                              // points v_begin elements BEFORE the shard's first element, so that
                              // token t of the whole vocabulary is element t of a row, and V is
                              // the shard's end
};

// element-wise masking of [begin, end) of one row; any alignment
template <typename E, bool ARGMAX>
__device__ __forceinline__ void apply_scalar(E *row, const uint32_t *mrow, int begin, int end,
                                             unsigned long long &best) {
    for (int t = begin + (int)threadIdx.x; t < end; t += APPLY_THREADS) {
        const bool keep = (mrow[t >> 5] >> (t & 31)) & 1u;
        if (!keep) {
            row[t] = (E)ElemTraits<E>::NEG_INF;
        } else if (ARGMAX) {
            const unsigned long long k = pack_best(order_key(ElemTraits<E>::f32_bits(row[t])), t);
            best = k > best ? k : best;
        }
    }
}

template <bool ARGMAX>
__device__ __forceinline__ void block_argmax_commit(unsigned long long best,
                                                    unsigned long long *dst) {
    if constexpr (ARGMAX) {
        __shared__ unsigned long long warp_best[APPLY_WARPS];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, best, o);
            best = other > best ? other : best;
        }
        if ((threadIdx.x & 31) == 0) warp_best[threadIdx.x >> 5] = best;
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 1; w < APPLY_WARPS; ++w) best = warp_best[w] > best ? warp_best[w] : best;
            if (best != 0ull) atomicMax(dst, best);
        }
    }
}

__device__ __forceinline__ __nv_bfloat162 as_bf162(uint32_t w) {
    return *reinterpret_cast<const __nv_bfloat162 *>(&w);
}
__device__ __forceinline__ uint32_t bf162_bits(__nv_bfloat162 v) {
    return *reinterpret_cast<const uint32_t *>(&v);
}

// Programmatic dependent launch: let the next kernel of the stream be scheduled early, then
// wait until the kernels before this one have finished and their writes are visible.  Both
// are no-ops for a kernel launched without the attribute.
__device__ __forceinline__ void pdl_enter() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// The two sweeps of the apply kernels over the spans [span_begin, span_end) of one row, for the
// calling block: this warp's spans are span_begin + warp, + APPLY_WARPS, ...; words[k] holds mask
// word `lane` of the k-th of them.  Returns the packed (value, token) maximum of this thread's
// allowed elements (0 when it saw none).
template <typename E, bool ARGMAX>
__device__ __forceinline__ unsigned long long apply_spans(E *row, const uint32_t (&words)[APPLY_SPANS_PER_WARP],
                                                          int span_begin, int span_end, int V) {
    constexpr int EPC = ElemTraits<E>::PER_CHUNK;  // elements per chunk: bits per lane
    constexpr int CHUNKS_PER_WORD = 32 / EPC;      // 4 (bf16) or 8 (fp32)
    constexpr int PASSES = CHUNKS_PER_WORD;        // 16-byte accesses per lane and span
    constexpr int GROUP = 4;                       // accesses issued together
    constexpr uint32_t FULL = (1u << EPC) - 1;
    constexpr uint32_t SKIP = 0xFFFFFFFFu;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int full_chunks = V / EPC;  // chunks that lie wholly inside the row
    // Per-lane running maximum: a strict float compare keeps the first of equal values and
    // treats -0.0 and +0.0 as equal; !(m <= best_v) also takes the very first candidate chunk,
    // whatever its value (best_v starts as NaN).
    float best_v = __uint_as_float(0x7FC00000u);
    int best_chunk = -1;
    uint32_t best_bits = 0, best_w[4] = {0, 0, 0, 0};

    // Sweep 1: every chunk whose bits are all clear is a pure store; chunks that will have to
    // be read (mixed bits, or any allowed element when the argmax is wanted) are only
    // prefetched into L2 here, so no warp waits on DRAM while its stores could be going out.
#pragma unroll
    for (int k = 0; k < APPLY_SPANS_PER_WARP; ++k) {
        const int span = span_begin + warp + k * APPLY_WARPS;
        if (span >= span_end) break;
        const int chunk0 = span * 32 * CHUNKS_PER_WORD;
#pragma unroll
        for (int p = 0; p < PASSES; ++p) {
            const int c = p * 32 + lane;  // chunk index inside the span
            const uint32_t word = __shfl_sync(0xFFFFFFFFu, words[k], c / CHUNKS_PER_WORD);
            const uint32_t bits = (word >> (EPC * (c % CHUNKS_PER_WORD))) & FULL;
            if (chunk0 + c >= full_chunks) continue;
            uint4 *ptr = reinterpret_cast<uint4 *>(row) + chunk0 + c;
            if (bits == 0) {
                const uint32_t ninf = sizeof(E) == 2 ? NEG_INF_BF16X2 : NEG_INF_F32;
                __stcs(ptr, make_uint4(ninf, ninf, ninf, ninf));
            } else if (ARGMAX || bits != FULL) {
                asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
            }
        }
    }
    // Sweep 2: the chunks that need their old contents, a group of independent loads at a time.
#pragma unroll
    for (int k = 0; k < APPLY_SPANS_PER_WARP; ++k) {
        const int span = span_begin + warp + k * APPLY_WARPS;
        if (span >= span_end) break;
        const int chunk0 = span * 32 * CHUNKS_PER_WORD;
        // a span without a single allowed token has nothing left to do (uniform per warp)
        if (__ballot_sync(0xFFFFFFFFu, words[k] != 0) == 0) continue;
#pragma unroll
        for (int p0 = 0; p0 < PASSES; p0 += GROUP) {
            uint4 val[GROUP];
            uint32_t bits[GROUP];
#pragma unroll
            for (int q = 0; q < GROUP; ++q) {
                const int c = (p0 + q) * 32 + lane;
                const uint32_t word = __shfl_sync(0xFFFFFFFFu, words[k], c / CHUNKS_PER_WORD);
                bits[q] = (word >> (EPC * (c % CHUNKS_PER_WORD))) & FULL;
                if (chunk0 + c >= full_chunks || bits[q] == 0 || (!ARGMAX && bits[q] == FULL))
                    bits[q] = SKIP;
                else
                    // a plain load, not a streaming one: a mixed chunk is stored back right
                    // away and should still find its line
                    val[q] = *(reinterpret_cast<const uint4 *>(row) + chunk0 + c);
            }
#pragma unroll
            for (int q = 0; q < GROUP; ++q) {
                if (bits[q] == SKIP) continue;
                const int chunk = chunk0 + (p0 + q) * 32 + lane;
                uint32_t w[4] = {val[q].x, val[q].y, val[q].z, val[q].w};
                if (bits[q] != FULL) {  // disallowed elements become -inf
                    if (sizeof(E) == 2) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            // one byte permute per pair: bytes 0-3 are the pair, 4-7 the two -inf;
                            // an allowed element takes its own bytes, a refused one those of -inf
                            const uint32_t two = (bits[q] >> (2 * i)) & 3u;
                            const uint32_t sel = 0x7654u - 0x0044u * (two & 1u) - 0x4400u * (two >> 1);
                            w[i] = __byte_perm(w[i], NEG_INF_BF16X2, sel);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            if (!((bits[q] >> i) & 1u)) w[i] = NEG_INF_F32;
                    }
                    __stcs(reinterpret_cast<uint4 *>(row) + chunk, make_uint4(w[0], w[1], w[2], w[3]));
                }
                if (ARGMAX) {
                    // The maximum of the chunk over the patched values (disallowed ones are -inf
                    // now) costs a few max instructions; the element is looked up only when it
                    // beats the lane's running maximum, which soon becomes rare.
                    float m;
                    if (sizeof(E) == 2) {
                        const __nv_bfloat162 m2 = __hmax2(__hmax2(as_bf162(w[0]), as_bf162(w[1])),
                                                          __hmax2(as_bf162(w[2]), as_bf162(w[3])));
                        const uint32_t u = bf162_bits(m2);
                        m = fmaxf(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
                    } else {
                        m = fmaxf(fmaxf(__uint_as_float(w[0]), __uint_as_float(w[1])),
                                  fmaxf(__uint_as_float(w[2]), __uint_as_float(w[3])));
                    }
                    // Only the chunk and its words are noted here (selects, no divergence: with a few
                    // chunks per lane nearly every warp would otherwise take the slow branch);
                    // the element is looked up once, after the loop.
                    const bool better = !(m <= best_v);
                    best_v = better ? m : best_v;
                    best_chunk = better ? chunk : best_chunk;
                    best_bits = better ? bits[q] : best_bits;
#pragma unroll
                    for (int i = 0; i < 4; ++i) best_w[i] = better ? w[i] : best_w[i];
                }
            }
        }
    }
    unsigned long long packed = 0ull;
    if (ARGMAX && best_chunk >= 0) {
        // the lane's winning chunk (as patched: disallowed elements are -inf there, but only
        // allowed ones count): the lowest allowed id that holds the maximum
        const uint32_t *w = best_w;
        int idx = -1;
#pragma unroll
        for (int i = EPC - 1; i >= 0; --i) {  // descending: the lowest id stays
            const uint32_t e = sizeof(E) == 2
                ? ((i & 1) ? (w[i >> 1] & 0xFFFF0000u) : (w[i >> 1] << 16)) : w[i];
            if (((best_bits >> i) & 1u) && __uint_as_float(e) == best_v) idx = best_chunk * EPC + i;
        }
        packed = pack_best(order_key(__float_as_uint(best_v)), idx);
    }
    return packed;
}

// grid = (blocks per row, B).  Requires 16-byte aligned rows (pointer and stride).
template <typename E, bool ARGMAX, bool GATHER>
// (every variant fits 64 registers, four blocks per SM; one of them has to be told)
__global__ void __launch_bounds__(APPLY_THREADS, (sizeof(E) == 4 && ARGMAX && !GATHER) ? 4 : 0)
apply_mask_kernel(ApplyArgs a, CtxDev ctx, unsigned long long *argkey) {
    constexpr int EPC = ElemTraits<E>::PER_CHUNK;  // elements per 16-byte chunk
    pdl_enter();
    const int r = blockIdx.y;
    E *row = static_cast<E *>(a.logits) + (int64_t)r * a.row_stride;
    const uint32_t *own = a.bitmask + (int64_t)r * a.mask_stride;
    const uint32_t *mrow = own;
    const uint2 *entry = nullptr;  // header row of the state's compact cache entry, if any
    bool entry_failed = false;     // no room in the arena: the staging row holds the mask
    if (GATHER) {
        const int32_t slot = ctx.slot[r];
        if (slot >= 0 && !ctx.compact) {
            mrow = ctx.pool + (int64_t)slot * ctx.pool_stride;
        } else if (slot >= 0) {
            // The entry is read without waiting for its failure flag (the header row of a cache
            // row in use only ever names stored words); a failed entry is read again below.
            entry = ctx.ent_hdr + (int64_t)slot * ctx.hdr_stride;
            entry_failed = ctx.ent_fail[slot] != 0;
            mrow = nullptr;
        }
    }
    const bool copy_out = GATHER && mrow != own;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_spans = (a.W + 31) / 32;
    const int span_begin = a.span_first + blockIdx.x * a.spans_per_block;
    const int span_end = min(span_begin + a.spans_per_block, n_spans);
    const int full_chunks = a.V / EPC;  // chunks that lie wholly inside the row
    // The mask words of every span this warp will handle are fetched first, so their L2
    // latency is paid once and not once per span (the spans themselves are store streams).
    uint32_t words[APPLY_SPANS_PER_WARP];
#pragma unroll
    for (int k = 0; k < APPLY_SPANS_PER_WARP; ++k) {
        const int w = (span_begin + warp + k * APPLY_WARPS) * 32 + lane;
        words[k] = 0;
        if (span_begin + warp + k * APPLY_WARPS < span_end) {
            if (GATHER && entry)
                words[k] = entry_word(entry, ctx.arena, span_begin + warp + k * APPLY_WARPS, lane,
                                      a.V, a.W);
            else if (w < a.W)
                words[k] = mrow[w];
        }
    }
    if (GATHER && entry_failed) {  // built in this call, no room in the arena (uniform per block)
        const uint32_t *srow = ctx.stage + (int64_t)ctx.ent_stage[ctx.slot[r]] * ctx.pool_stride;
#pragma unroll
        for (int k = 0; k < APPLY_SPANS_PER_WARP; ++k) {
            const int w = (span_begin + warp + k * APPLY_WARPS) * 32 + lane;
            if (span_begin + warp + k * APPLY_WARPS < span_end && w < a.W) words[k] = srow[w];
        }
    }
    if (copy_out) {
#pragma unroll
        for (int k = 0; k < APPLY_SPANS_PER_WARP; ++k) {
            const int w = (span_begin + warp + k * APPLY_WARPS) * 32 + lane;
            if (span_begin + warp + k * APPLY_WARPS < span_end && w < a.W)
                a.bitmask_out[(int64_t)r * a.mask_stride + w] = words[k];
        }
    }
    unsigned long long packed = apply_spans<E, ARGMAX>(row, words, span_begin, span_end, a.V);
    // elements after the last whole chunk (V not a multiple of the chunk size)
    if (blockIdx.x == gridDim.x - 1 && full_chunks * EPC < a.V) {
        if (GATHER && entry) {  // the row's last words were written out by this very block
            __syncthreads();
            mrow = own;
        }
        apply_scalar<E, ARGMAX>(row, mrow, full_chunks * EPC, a.V, packed);
    }
    block_argmax_commit<ARGMAX>(packed, argkey + r);
}

// Any alignment: one block column per row, element-wise.
template <typename E, bool ARGMAX, bool GATHER>
__global__ void __launch_bounds__(APPLY_THREADS)
apply_mask_unaligned_kernel(ApplyArgs a, CtxDev ctx, unsigned long long *argkey) {
    pdl_enter();
    const int r = blockIdx.y;
    E *row = static_cast<E *>(a.logits) + (int64_t)r * a.row_stride;
    const uint32_t *own = a.bitmask + (int64_t)r * a.mask_stride;
    const uint32_t *mrow = own;
    const int t_first = a.span_first * 1024;
    const int per_block = ((a.V - t_first + gridDim.x - 1) / gridDim.x + 31) & ~31;
    const int begin = t_first + blockIdx.x * per_block, end = min(begin + per_block, a.V);
    if (GATHER) {
        const int32_t slot = ctx.slot[r];
        if (slot >= 0 && !ctx.compact) {
            mrow = ctx.pool + (int64_t)slot * ctx.pool_stride;
        } else if (slot >= 0) {
            if (ctx.ent_fail[slot]) {
                mrow = ctx.stage + (int64_t)ctx.ent_stage[slot] * ctx.pool_stride;
            } else if (begin < end) {
                // expand the block's words of the compact entry into the row's own bitmask,
                // then mask from there
                const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
                const int w_begin = begin >> 5, w_end = (end + 31) >> 5;
                const uint2 *hdr_row = ctx.ent_hdr + (int64_t)slot * ctx.hdr_stride;
                for (int span = (w_begin >> 5) + warp; span * 32 < w_end; span += APPLY_WARPS) {
                    const uint32_t word = entry_word(hdr_row, ctx.arena, span, lane, a.V, a.W);
                    const int w = span * 32 + lane;
                    if (w >= w_begin && w < w_end) a.bitmask_out[(int64_t)r * a.mask_stride + w] = word;
                }
                __syncthreads();
            }
        }
    }
    if (GATHER && mrow != own)
        for (int i = (begin >> 5) + (int)threadIdx.x; i < (end + 31) >> 5; i += APPLY_THREADS)
            a.bitmask_out[(int64_t)r * a.mask_stride + i] = mrow[i];
    unsigned long long best = 0ull;
    if (begin < end) apply_scalar<E, ARGMAX>(row, mrow, begin, end, best);
    block_argmax_commit<ARGMAX>(best, argkey + r);
}

__global__ void argmax_finish_kernel(const unsigned long long *argkey, int B, int32_t *out) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < B) out[r] = unpack_best(argkey[r]);
}

// ---------------------------------------------------------------------------------------
// K6: advance.  One thread per row; at most a handful of dependent lookups.
// from_keys: the token comes from the packed maxima of the fused step and is written out.
// ---------------------------------------------------------------------------------------
// Packed maxima leave the library as signed 64-bit integers whose signed order is the order of
// the packed keys (top bit flipped), so that an all-reduce with MAX over ranks picks the winner.
__device__ __forceinline__ long long key_to_signed(unsigned long long k) {
    return (long long)(k ^ 0x8000000000000000ull);
}
__device__ __forceinline__ unsigned long long key_from_signed(long long k) {
    return (unsigned long long)k ^ 0x8000000000000000ull;
}

// The fused step's packed maxima out to the caller, and zeroed for the next step.
__global__ void export_keys_kernel(CtxDev ctx, long long *out, int B) {
    pdl_enter();
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= B) return;
    out[r] = key_to_signed(ctx.argkey[r]);
    ctx.argkey[r] = 0ull;
}

// Row r takes token t: the new state into sid[r], the row's status out.  `chosen`: the token is
// the step's own greedy choice (-1 = nothing was allowed).
__device__ __forceinline__ void advance_row(const VocabDev &v, const CtxDev &ctx, const GrammarDev &gr,
                                            bool known, int32_t *sid, int32_t *status, uint32_t flags,
                                            int r, int t, bool chosen) {
    const uint32_t s = (uint32_t)sid[r];
    int32_t st = WG_OK;
    if (!known || s >= (uint32_t)gr.n_states) {
        st = WG_ERR_STATE;
        atomicAdd(&ctx.stats[ST_BAD_STATE], 1ull);
    } else if (chosen && t < 0) {
        st = WG_ERR_EMPTY_MASK;
        atomicAdd(&ctx.stats[ST_EMPTY], 1ull);
    } else {
        uint32_t next = 0;
        if (gr.forced && s != 0 && gr.forced[s].x >= 0) {  // token-level Write: that token only
            const int2 f = gr.forced[s];
            if (t == f.x && t < v.V) next = (uint32_t)f.y;
        } else if (t >= 0 && t < v.V && s != 0) {
            // the class-mapped record of the token: one dependent look-up per byte instead of
            // two (this is a chain of dependent loads at the very end of every step)
            if (t == v.eos_id)
                next = gr.wide ? static_cast<const uint32_t *>(gr.table)[(size_t)s * gr.n_classes + gr.eos_class]
                               : static_cast<const uint16_t *>(gr.table)[(size_t)s * gr.n_classes + gr.eos_class];
            else
                next = gr.wide
                    ? walk_token_classes<uint32_t>(v, gr.rec_class, static_cast<const uint32_t *>(gr.table),
                                                   gr.n_classes, gr.byte_class, s, t)
                    : walk_token_classes<uint16_t>(v, gr.rec_class, static_cast<const uint16_t *>(gr.table),
                                                   gr.n_classes, gr.byte_class, s, t);
        }
        if (next == 0) {
            st = WG_ERR_TOKEN_REJECTED;
            atomicAdd(&ctx.stats[ST_REJECTED], 1ull);
        } else {
            if ((flags & WG_RESTART_ON_DONE) && next == (uint32_t)gr.done) next = (uint32_t)gr.start;
            sid[r] = (int32_t)next;
        }
    }
    if (status) status[r] = st;
}

// from_keys: 0 = the tokens come in token_in; 1 = from the fused step's packed maxima; 2 = from
// ext_keys (signed packed maxima, e.g. after an all-reduce over vocabulary shards).
__global__ void advance_kernel(VocabDev v, CtxDev ctx, const int32_t *gid, int32_t *sid,
                               const int32_t *token_in, int32_t *token_out, int B,
                               int32_t *status, uint32_t flags, int from_keys,
                               const long long *ext_keys) {
    // What never changes while steps are in flight (the row's grammar id, the grammar's record)
    // is read BEFORE waiting for the kernel ahead, so that these two dependent loads run under
    // its tail; states and tokens are only touched after the wait.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    const int g = r < B ? gid[r] : -1;
    const bool known = g >= 0 && g < ctx.n_grammars;
    GrammarDev gr = {};
    if (known) gr = ctx.grammars[g];
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (r >= B) return;
    int t;
    if (from_keys == 2) {
        t = unpack_best(key_from_signed(ext_keys[r]));
        token_out[r] = t;
    } else if (from_keys) {
        t = unpack_best(ctx.argkey[r]);
        ctx.argkey[r] = 0ull;  // ready for the next step
        token_out[r] = t;
    } else {
        t = token_in[r];
    }
    advance_row(v, ctx, gr, known, sid, status, flags, r, t, from_keys != 0);
}

// ---------------------------------------------------------------------------------------
// The whole decode step of a SMALL batch in one launch.  With a handful of rows the four kernels
// of the step cost more in launches and in the waits between them than in work, so here every
// block does everything for its part of a row: it probes the cache itself (all blocks of a row
// make the same read-only probe), takes the mask words from the cached row or, on a miss, builds
// the words of its own spans (the warp-level build above), masks and scans its logits, and the
// block that finishes a row LAST (a per-row arrival counter) advances the row's state and, after
// a miss, files the finished mask row in the cache.  Rows that meet the same new state in one
// step each build it (there are few rows); one of them files it.
// grid = (blocks per row, B); needs 16-byte aligned rows.
// ---------------------------------------------------------------------------------------
struct SmallStepArgs {
    const int32_t *gid;
    int32_t *sid;        // in / out
    int32_t *token_out;
    int32_t *status;     // or NULL
    uint32_t flags;      // WG_RESTART_ON_DONE or 0
    int32_t use_cache;   // 0: WG_NO_CACHE (every row is built, nothing is probed or filed)
};

template <typename E>
__global__ void __launch_bounds__(APPLY_THREADS)
decode_step_small_kernel(ApplyArgs a, CtxDev ctx, VocabDev v, SmallStepArgs st) {
    constexpr int EPC = ElemTraits<E>::PER_CHUNK;
    constexpr int K = APPLY_SPANS_PER_WARP;
    __shared__ MaskFacts facts;
    __shared__ uint16_t queues[APPLY_WARPS][WARP_QUEUE];
    __shared__ uint32_t scratch[APPLY_WARPS][K * 32];
    __shared__ int32_t sh_slot, sh_last, sh_new_row;
    pdl_enter();
    const int r = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    E *row = static_cast<E *>(a.logits) + (int64_t)r * a.row_stride;
    uint32_t *own = a.bitmask_out + (int64_t)r * a.mask_stride;
    const int g = st.gid[r], s = st.sid[r];
    // ---- where the row's mask comes from
    if (threadIdx.x == 0) {
        int32_t slot = -1;
        if (st.use_cache && g >= 0 && g < ctx.n_grammars && s > 0 && s < ctx.grammars[g].n_states)
            slot = cache_probe(ctx, g, s);          // -1: not cached, -2: cached without a row
        sh_slot = slot;
        if (blockIdx.x == 0) {
            if (slot >= 0) atomicAdd(&ctx.stats[ST_HITS], 1ull);
            else if (st.use_cache) atomicAdd(&ctx.stats[ST_MISSES], 1ull);
        }
    }
    __syncthreads();
    const int32_t slot = sh_slot;
    const int n_spans = (a.W + 31) / 32;
    const int span_begin = a.span_first + blockIdx.x * a.spans_per_block;
    const int span_end = min(span_begin + a.spans_per_block, n_spans);
    uint32_t words[K];
    if (slot >= 0) {
        const bool failed = ctx.compact && ctx.ent_fail[slot] != 0;   // (never true: probed above)
        const uint2 *entry = ctx.compact ? ctx.ent_hdr + (int64_t)slot * ctx.hdr_stride : nullptr;
        const uint32_t *mrow = ctx.compact ? nullptr : ctx.pool + (int64_t)slot * ctx.pool_stride;
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const int span = span_begin + warp + k * APPLY_WARPS;
            const int w = span * 32 + lane;
            words[k] = 0;
            if (span < span_end && !failed) {
                if (entry) words[k] = entry_word(entry, ctx.arena, span, lane, a.V, a.W);
                else if (w < a.W) words[k] = mrow[w];
            }
        }
    } else {
        // ---- build this block's spans of the mask
        if (warp == 0) gather_item_facts(v, ctx, g, s, own, -1, blockIdx.x == 0, facts);
        __syncthreads();
        uint16_t *queue = queues[warp];
        uint32_t *mine = scratch[warp];
#pragma unroll
        for (int k = 0; k < K; ++k) mine[k * 32 + lane] = 0u;
        int w[K];
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const int span = span_begin + warp + k * APPLY_WARPS;
            w[k] = (span < span_end && span * 32 + lane < a.W) ? span * 32 + lane : -1;
        }
        uint32_t alive[K], todo[K];
        int unused_a = 0, unused_b = 0;
        decide_words<K, false>(v, facts, w, alive, todo, unused_a);
        const int t_base = (span_begin + warp) << 10;
        int n_todo = 0;
#pragma unroll
        for (int k = 0; k < K; ++k) n_todo += __popc(todo[k]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) n_todo += __shfl_xor_sync(0xFFFFFFFFu, n_todo, o);
        if (n_todo > WARP_QUEUE) {   // a state that walks most tokens: span by span
#pragma unroll
            for (int k = 0; k < K; ++k) {
                const int n = push_queued<K>(queue, 0, todo, 1u << k);
                walk_queued<false>(v, facts, queue, n, t_base, APPLY_WARPS << 10, mine, unused_b);
            }
        } else if (n_todo > 0) {
            const int n = push_queued<K>(queue, 0, todo, (1u << K) - 1u);
            walk_queued<false>(v, facts, queue, n, t_base, APPLY_WARPS << 10, mine, unused_b);
        } else {
            __syncwarp();
        }
#pragma unroll
        for (int k = 0; k < K; ++k) words[k] = alive[k] | mine[k * 32 + lane];
    }
    // ---- the row's mask words out, then mask and scan the logits
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const int span = span_begin + warp + k * APPLY_WARPS;
        const int w = span * 32 + lane;
        if (span < span_end && w < a.W) own[w] = words[k];
    }
    unsigned long long packed = apply_spans<E, true>(row, words, span_begin, span_end, a.V);
    const int full_chunks = a.V / EPC;
    if (blockIdx.x == gridDim.x - 1 && full_chunks * EPC < a.V) {
        __syncthreads();   // the row's last words were written out by this very block
        apply_scalar<E, true>(row, own, full_chunks * EPC, a.V, packed);
    }
    block_argmax_commit<true>(packed, ctx.argkey + r);
    // ---- the last block of the row ends the step for it
    if (threadIdx.x == 0) {
        __threadfence();
        sh_last = atomicAdd(&ctx.row_done[r], 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (!sh_last) return;
    __threadfence();
    if (threadIdx.x == 0) {
        ctx.row_done[r] = 0;
        const int t = unpack_best(atomicExch(&ctx.argkey[r], 0ull));   // zero again for the next step
        st.token_out[r] = t;
        const bool known = g >= 0 && g < ctx.n_grammars;
        GrammarDev gr = {};
        if (known) gr = ctx.grammars[g];
        // File the mask first: the key is claimed here, the row index published after the copy.
        // A built row that nobody files (no cache, no room, a state the grammar does not have)
        // counts as uncached.
        int32_t new_row = -1;
        if (st.use_cache && slot < 0) {
            bool filed = false;   // by this row, or by another row that met the same state
            if (ctx.hash_size > 0 && known && s > 0 && s < gr.n_states) {
                const unsigned long long key = cache_key(g, s);
                const uint32_t mask = (uint32_t)ctx.hash_size - 1;
                uint32_t h = cache_hash(key) & mask;
                for (int probe = 0; probe < ctx.hash_size; ++probe, h = (h + 1) & mask) {
                    unsigned long long k = ctx.keys[h];
                    if (k == 0) {
                        if (pool_full(ctx)) break;
                        k = atomicCAS(&ctx.keys[h], 0ull, key);
                        if (k == 0) {
                            const int32_t got = take_pool_row(ctx);
                            if (got >= 0) {        // (else the key stays, without a row)
                                new_row = got;
                                filed = true;
                                if (ctx.compact) ctx.ent_fail[got] = 0;
                            }
                            ctx.ent[r] = (int32_t)h;
                            break;
                        }
                    }
                    if (k == key) {
                        // another row files it in this step (or did, with a compact entry that
                        // found no room); a key left without a row by a full pool is not filed
                        filed = !pool_full(ctx) || *(volatile int32_t *)&ctx.vals[h] >= 0;
                        break;
                    }
                }
            }
            if (!filed) atomicAdd(&ctx.stats[ST_UNCACHED], 1ull);
        }
        sh_new_row = new_row;
        advance_row(v, ctx, gr, known, st.sid, st.status, st.flags, r, t, true);
    }
    __syncthreads();
    const int32_t new_row = sh_new_row;
    if (new_row < 0) return;
    if (!ctx.compact) {
        uint32_t *dst = ctx.pool + (int64_t)new_row * ctx.pool_stride;
        for (int w = threadIdx.x; w < a.W; w += APPLY_THREADS) dst[w] = __ldcg(&own[w]);
    } else {
        for (int span = warp; span < n_spans; span += APPLY_WARPS) {
            const int w = span * 32 + lane;
            store_span(ctx.ent_hdr + (int64_t)new_row * ctx.hdr_stride, ctx.arena, ctx.arena_top,
                       ctx.arena_words, ctx.ent_fail + new_row, ctx.stats + ST_UNCACHED, span,
                       w < a.W ? __ldcg(&own[w]) : 0u, lane, a.V, a.W);
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) ctx.vals[ctx.ent[r]] = new_row;   // from now on a probe finds the row
}
