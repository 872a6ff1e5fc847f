// Host side of the C ABI declared in wg.h: object lifetimes, uploads and kernel launches.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "wg_kernels.cuh"

namespace {

// NVTX range around an entry point, so that a timeline shows the calls by name (costs a few
// nanoseconds when no profiler is attached).
struct NvtxRange {
    explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
};

thread_local int32_t g_last_cuda_error = 0;
std::atomic<int64_t> g_launches{0};

#define WG_CUDA(expr)                                   \
    do {                                                \
        cudaError_t e__ = (expr);                       \
        if (e__ != cudaSuccess) {                       \
            g_last_cuda_error = (int32_t)e__;           \
            return WG_ERR_CUDA;                         \
        }                                               \
    } while (0)

// after a <<< >>> launch: count it and pick up a launch-configuration error
#define WG_LAUNCHED()                                   \
    do {                                                \
        g_launches.fetch_add(1, std::memory_order_relaxed); \
        WG_CUDA(cudaGetLastError());                    \
    } while (0)

int g_sm_count = 0;
int sm_count() {
    if (g_sm_count == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
            g_sm_count = n;
        else
            g_sm_count = 148;
    }
    return g_sm_count;
}

// Launch with programmatic stream serialization: the kernel may be scheduled while the
// kernel before it in the stream is still running; it orders itself with griddepcontrol.wait.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st,
                       Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <typename T>
int32_t dev_alloc(T **p, size_t n) {
    *p = nullptr;
    WG_CUDA(cudaMalloc((void **)p, (n ? n : 1) * sizeof(T)));
    return WG_OK;
}

}  // namespace

struct wg_vocab {
    VocabDev dev{};
    void *d_rec = nullptr, *d_len = nullptr, *d_offsets = nullptr, *d_bytes = nullptr;
    void *d_first_mask = nullptr, *d_fold_mask = nullptr, *d_valid_mask = nullptr;
    int device = 0;
};

struct GrammarSlot {
    uint64_t hash;
    std::vector<int32_t> table;  // host copy, for exact comparison on hash equality
    std::vector<int32_t> forced_tok, forced_next;
    int32_t n_states, n_classes;
    void *d_table, *d_cls, *d_first_ok, *d_leaves, *d_forced, *d_leave1, *d_leave_fold;
    // the rest of what makes two grammars the same: equal tables over different class maps
    // (Write("a") and Write("b")) are different grammars
    uint8_t byte_class[256];
    int32_t start, done, eos_class;
    bool removed = false;  // wg_ctx_remove_grammar: the id waits to be given to another grammar

    bool same_as(const wg_grammar &g) const {
        return !removed && hash == g.hash && n_states == g.n_states && n_classes == g.n_classes &&
               start == g.start && done == g.done && eos_class == g.eos_class &&
               memcmp(byte_class, g.byte_class, 256) == 0 && table == g.table &&
               forced_tok == g.forced_tok && forced_next == g.forced_next;
    }
};

struct ClassMappedRecords {
    uint8_t byte_class[256];
    void *d_rec;  // uint4[V]
    int users;    // grammars of the context that walk these records
};

struct wg_ctx {
    const wg_vocab *vocab = nullptr;
    std::vector<ClassMappedRecords> class_records;  // one per distinct byte_class map
    CtxDev dev{};
    std::vector<GrammarDev> grammars;  // host mirror of dev.grammars
    std::vector<GrammarSlot> slots;
    GrammarDev *d_grammars = nullptr;
    int32_t grammar_cap = 0;
    int32_t max_batch = 0;
    // vocabulary-sharded steps fill cached masks only inside their token range; the range they
    // used is remembered so that no call reads cached words that were never built
    int32_t part_begin = 0, part_end = 0;  // both 0: every cached mask is complete
    int build_blocks_per_sm = 0;           // resident blocks of the build kernel (0: not asked yet)
    // "what follows byte b" masks (see after_masks_kernel): made on demand, at most AFTER_SLOTS bytes
    uint32_t *d_after_masks = nullptr;
    int8_t *d_after_slot = nullptr;
    uint32_t *d_leave_bits = nullptr;      // 8 words of scratch for wg_ctx_add_grammar
    int8_t after_slot[256];
    int n_after = 0;
    int32_t *d_stage_gid = nullptr, *d_stage_sid = nullptr;  // prewarm staging
    std::vector<void *> owned;  // every other device allocation
    std::mutex mu;
    bool count_build_work = false;  // launch the counting variant of the build kernel
    int64_t removed_keys = 0;       // hash-table entries of removed grammars still in the table
    int32_t *d_counts = nullptr;    // scratch of wg_ctx_remove_grammar
    // optional per-kernel timing: events[4 * i + {0,1,2,3}] = build begin/end, apply begin/end
    bool timing = false;
    std::vector<cudaEvent_t> events;
    size_t timed_steps = 0;
};

namespace {
constexpr size_t MAX_TIMED_STEPS = 8192;

// Records event `which` (0..3) of the current timed step; grows the event pool on demand.
int32_t timing_mark(wg_ctx *c, int which, cudaStream_t st) {
    if (!c->timing || c->timed_steps >= MAX_TIMED_STEPS) return WG_OK;
    const size_t idx = 4 * c->timed_steps + (size_t)which;
    while (c->events.size() <= idx) {
        cudaEvent_t e;
        WG_CUDA(cudaEventCreate(&e));
        c->events.push_back(e);
    }
    WG_CUDA(cudaEventRecord(c->events[idx], st));
    if (which == 3) ++c->timed_steps;
    return WG_OK;
}
}  // namespace

extern "C" {

const char *wg_strerror(int32_t status) {
    switch (status) {
    case WG_OK: return "ok";
    case WG_ERR_ARG: return "bad argument";
    case WG_ERR_GRAMMAR: return "operator tree breaks a grammar rule";
    case WG_ERR_CAPACITY: return "capacity exhausted (a fixed-size table or scratch array is too small)";
    case WG_ERR_TOKEN_REJECTED: return "token not allowed in this state";
    case WG_ERR_CUDA: return "CUDA runtime error";
    case WG_ERR_EMPTY_MASK: return "no token allowed";
    case WG_ERR_STATE: return "grammar or state id out of range";
    default: return "unknown status";
    }
}

int32_t wg_last_cuda_error(void) { return g_last_cuda_error; }
int64_t wg_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

// ---- vocabulary ---------------------------------------------------------------------

int32_t wg_load_vocab(const uint32_t *offsets, const uint8_t *bytes, int32_t V, int32_t eos_id,
                      wg_vocab **out) {
    NvtxRange nvtx_range("wg_load_vocab");
    if (!out) return WG_ERR_ARG;
    *out = nullptr;
    if (!offsets || V <= 0 || eos_id < 0 || eos_id >= V || offsets[0] != 0) return WG_ERR_ARG;
    for (int32_t t = 0; t < V; ++t)
        if (offsets[t + 1] < offsets[t]) return WG_ERR_ARG;
    const uint32_t total = offsets[V];
    if (total > 0 && !bytes) return WG_ERR_ARG;

    std::vector<uint8_t> rec((size_t)V * WG_REC_BYTES, 0), len(V, 0);
    // V-bit masks used by the build kernel: starts-with-byte (256), contains-a-byte-folding-to
    // (64), has-any-byte (1); W words each
    const size_t W = ((size_t)V + 31) / 32;
    std::vector<uint32_t> first_mask(256 * W, 0u), fold_mask(64 * W, 0u), valid_mask(W, 0u);
    for (int32_t t = 0; t < V; ++t) {
        const uint32_t n = (t == eos_id) ? 0u : offsets[t + 1] - offsets[t];
        len[t] = (uint8_t)(n > 255u ? 255u : n);
        if (!n) continue;
        const uint8_t *b = bytes + offsets[t];
        memcpy(&rec[(size_t)t * WG_REC_BYTES], b, n < WG_REC_BYTES ? n : WG_REC_BYTES);
        const uint32_t bit = 1u << (t & 31);
        const size_t w = (size_t)t >> 5;
        valid_mask[w] |= bit;
        first_mask[(size_t)b[0] * W + w] |= bit;
        for (uint32_t i = 0; i < n; ++i) fold_mask[(size_t)(b[i] & 63) * W + w] |= bit;
    }
    wg_vocab *v = new (std::nothrow) wg_vocab();
    if (!v) return WG_ERR_ARG;
    auto fail = [&](int32_t rc) { wg_vocab_free(v); return rc; };
    if (cudaGetDevice(&v->device) != cudaSuccess) return fail(WG_ERR_CUDA);
    if (cudaMalloc(&v->d_rec, rec.size()) != cudaSuccess ||
        cudaMalloc(&v->d_len, len.size()) != cudaSuccess ||
        cudaMalloc(&v->d_first_mask, first_mask.size() * sizeof(uint32_t)) != cudaSuccess ||
        cudaMalloc(&v->d_fold_mask, fold_mask.size() * sizeof(uint32_t)) != cudaSuccess ||
        cudaMalloc(&v->d_valid_mask, valid_mask.size() * sizeof(uint32_t)) != cudaSuccess ||
        cudaMalloc(&v->d_offsets, sizeof(uint32_t) * ((size_t)V + 1)) != cudaSuccess ||
        cudaMalloc(&v->d_bytes, total ? total : 1) != cudaSuccess)
        return fail(WG_ERR_CUDA);
    if (cudaMemcpy(v->d_rec, rec.data(), rec.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(v->d_len, len.data(), len.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(v->d_first_mask, first_mask.data(), first_mask.size() * sizeof(uint32_t),
                   cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(v->d_fold_mask, fold_mask.data(), fold_mask.size() * sizeof(uint32_t),
                   cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(v->d_valid_mask, valid_mask.data(), valid_mask.size() * sizeof(uint32_t),
                   cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(v->d_offsets, offsets, sizeof(uint32_t) * ((size_t)V + 1),
                   cudaMemcpyHostToDevice) != cudaSuccess ||
        (total && cudaMemcpy(v->d_bytes, bytes, total, cudaMemcpyHostToDevice) != cudaSuccess))
        return fail(WG_ERR_CUDA);
    v->dev.rec = static_cast<const uint4 *>(v->d_rec);
    v->dev.len = static_cast<const uint8_t *>(v->d_len);
    v->dev.first_mask = static_cast<const uint32_t *>(v->d_first_mask);
    v->dev.fold_mask = static_cast<const uint32_t *>(v->d_fold_mask);
    v->dev.valid_mask = static_cast<const uint32_t *>(v->d_valid_mask);
    v->dev.offsets = static_cast<const uint32_t *>(v->d_offsets);
    v->dev.bytes = static_cast<const uint8_t *>(v->d_bytes);
    v->dev.V = V;
    v->dev.W = (V + 31) / 32;
    v->dev.eos_id = eos_id;
    *out = v;
    return WG_OK;
}

void wg_vocab_free(wg_vocab *v) {
    if (!v) return;
    cudaFree(v->d_rec);
    cudaFree(v->d_len);
    cudaFree(v->d_first_mask);
    cudaFree(v->d_fold_mask);
    cudaFree(v->d_valid_mask);
    cudaFree(v->d_offsets);
    cudaFree(v->d_bytes);
    delete v;
}

// ---- grammars -----------------------------------------------------------------------

int32_t wg_compile_grammar(const wg_op_node *nodes, int32_t n_nodes, const int32_t *children,
                           int32_t n_children, const uint32_t *sets, int32_t n_sets,
                           const uint8_t *data, int32_t n_data, int32_t root, wg_grammar **out) {
    NvtxRange nvtx_range("wg_compile_grammar");
    if (!out) return WG_ERR_ARG;
    *out = nullptr;
    wg_grammar *g = new (std::nothrow) wg_grammar();
    if (!g) return WG_ERR_ARG;
    int32_t rc;
    try {
        rc = wg_lower_tree(nodes, n_nodes, children, n_children, sets, n_sets, data, n_data, root, g);
    } catch (const std::bad_alloc &) {
        rc = WG_ERR_CAPACITY;
    }
    if (rc != WG_OK) {
        delete g;
        return rc;
    }
    *out = g;
    return WG_OK;
}

void wg_grammar_free(wg_grammar *g) { delete g; }

int32_t wg_template_compile(const wg_op_node *nodes, int32_t n_nodes, const int32_t *children,
                            int32_t n_children, const uint32_t *sets, int32_t n_sets,
                            const uint8_t *data, int32_t n_data, int32_t root, wg_template **out) {
    NvtxRange nvtx_range("wg_template_compile");
    if (!out) return WG_ERR_ARG;
    *out = nullptr;
    wg_template *t = new (std::nothrow) wg_template();
    if (!t) return WG_ERR_ARG;
    int32_t rc;
    try {
        rc = wg_lower_tree(nodes, n_nodes, children, n_children, sets, n_sets, data, n_data, root,
                           &t->base, &t->sites);
        if (rc == WG_OK)  // every HOLE node counts, also one that no path reaches
            for (int32_t i = 0; i < n_nodes; ++i)
                if (nodes[i].kind == WG_OP_HOLE && nodes[i].reserved + 1 > t->n_args)
                    t->n_args = nodes[i].reserved + 1;
    } catch (const std::bad_alloc &) {
        rc = WG_ERR_CAPACITY;
    }
    if (rc != WG_OK) {
        delete t;
        return rc;
    }
    *out = t;
    return WG_OK;
}

int32_t wg_template_info(const wg_template *t, int32_t *n_states, int32_t *n_holes, int32_t *n_args) {
    if (!t) return WG_ERR_ARG;
    if (n_states) *n_states = t->base.n_states;
    if (n_holes) *n_holes = (int32_t)t->sites.size();
    if (n_args) *n_args = t->n_args;
    return WG_OK;
}

int32_t wg_template_instantiate(const wg_template *t, const wg_grammar *const *args, int32_t n_args,
                                wg_grammar **out) {
    NvtxRange nvtx_range("wg_template_instantiate");
    if (!out) return WG_ERR_ARG;
    *out = nullptr;
    if (!t) return WG_ERR_ARG;
    wg_grammar *g = new (std::nothrow) wg_grammar();
    if (!g) return WG_ERR_ARG;
    int32_t rc;
    try {
        rc = wg_instantiate_template(*t, args, n_args, g);
    } catch (const std::bad_alloc &) {
        rc = WG_ERR_CAPACITY;
    }
    if (rc != WG_OK) {
        delete g;
        return rc;
    }
    *out = g;
    return WG_OK;
}

void wg_template_free(wg_template *t) { delete t; }

int32_t wg_grammar_minimize(const wg_grammar *g, wg_grammar **out) {
    if (!g || !out) return WG_ERR_ARG;
    *out = nullptr;
    wg_grammar *m = new (std::nothrow) wg_grammar();
    if (!m) return WG_ERR_ARG;
    int32_t rc;
    try {
        rc = wg_minimize_grammar(*g, m);
    } catch (const std::bad_alloc &) {
        rc = WG_ERR_CAPACITY;
    }
    if (rc != WG_OK) {
        delete m;
        return rc;
    }
    *out = m;
    return WG_OK;
}

namespace {
constexpr uint32_t BLOB_MAGIC = 0x31474757u;  // "WGG1"
struct BlobHeader {
    uint32_t magic, version;
    int32_t n_states, n_classes, start, done, eos_class, has_forced, tail, reserved;
    uint64_t hash;
};
}  // namespace

int32_t wg_grammar_save(const wg_grammar *g, void *blob, size_t capacity, size_t *needed) {
    if (!g || !needed) return WG_ERR_ARG;
    const size_t n_table = g->table.size() * sizeof(int32_t);
    const size_t n_forced = g->forced_tok.size() * sizeof(int32_t);
    const size_t total = sizeof(BlobHeader) + 256 + n_table + 2 * n_forced;
    *needed = total;
    if (capacity < total || !blob) return WG_ERR_CAPACITY;
    uint8_t *p = static_cast<uint8_t *>(blob);
    const BlobHeader h{BLOB_MAGIC, 2u, g->n_states, g->n_classes, g->start, g->done, g->eos_class,
                       g->forced_tok.empty() ? 0 : 1, g->tail, 0, g->hash};
    memcpy(p, &h, sizeof(h)); p += sizeof(h);
    memcpy(p, g->byte_class, 256); p += 256;
    memcpy(p, g->table.data(), n_table); p += n_table;
    if (n_forced) {
        memcpy(p, g->forced_tok.data(), n_forced); p += n_forced;
        memcpy(p, g->forced_next.data(), n_forced);
    }
    return WG_OK;
}

int32_t wg_grammar_load(const void *blob, size_t size, wg_grammar **out) {
    if (!out) return WG_ERR_ARG;
    *out = nullptr;
    if (!blob || size < sizeof(BlobHeader) + 256) return WG_ERR_ARG;
    const uint8_t *p = static_cast<const uint8_t *>(blob);
    BlobHeader h;
    memcpy(&h, p, sizeof(h)); p += sizeof(h);
    if (h.magic != BLOB_MAGIC || h.version != 2u) return WG_ERR_ARG;
    if (h.tail < -1 || h.tail == 0 || h.tail >= h.n_states) return WG_ERR_ARG;
    if (h.n_states < 2 || h.n_classes < 1 || h.n_classes > WG_N_SYMBOLS) return WG_ERR_ARG;
    if (h.start < 1 || h.start >= h.n_states || h.done < 1 || h.done >= h.n_states ||
        h.eos_class < 0 || h.eos_class >= h.n_classes)
        return WG_ERR_ARG;
    const size_t cells = (size_t)h.n_states * (size_t)h.n_classes;
    const size_t n_forced = h.has_forced ? (size_t)h.n_states * sizeof(int32_t) : 0;
    if (size != sizeof(BlobHeader) + 256 + cells * sizeof(int32_t) + 2 * n_forced) return WG_ERR_ARG;
    wg_grammar *g = new (std::nothrow) wg_grammar();
    if (!g) return WG_ERR_ARG;
    bool ok = true;
    try {
        g->n_states = h.n_states; g->n_classes = h.n_classes; g->start = h.start; g->done = h.done;
        g->eos_class = h.eos_class; g->hash = h.hash; g->tail = h.tail;
        memcpy(g->byte_class, p, 256); p += 256;
        for (int b = 0; b < 256 && ok; ++b) ok = g->byte_class[b] < h.n_classes;
        g->table.resize(cells);
        memcpy(g->table.data(), p, cells * sizeof(int32_t)); p += cells * sizeof(int32_t);
        for (size_t i = 0; i < cells && ok; ++i) ok = g->table[i] >= 0 && g->table[i] < h.n_states;
        for (int32_t c = 0; c < h.n_classes && ok; ++c) ok = g->table[c] == 0;  // DEAD stays dead
        if (n_forced) {
            g->forced_tok.resize(h.n_states);
            g->forced_next.resize(h.n_states);
            memcpy(g->forced_tok.data(), p, n_forced); p += n_forced;
            memcpy(g->forced_next.data(), p, n_forced);
            for (int32_t st = 0; st < h.n_states && ok; ++st)
                ok = g->forced_tok[st] >= -1 && g->forced_next[st] >= 0 && g->forced_next[st] < h.n_states;
        }
    } catch (const std::bad_alloc &) {
        ok = false;
    }
    // the stored hash must be the hash of what was stored: grammars are told apart by it
    if (ok && wg_grammar_content_hash(*g) != h.hash) ok = false;
    if (!ok) {
        delete g;
        return WG_ERR_ARG;
    }
    *out = g;
    return WG_OK;
}

int32_t wg_grammar_info(const wg_grammar *g, int32_t *n_states, int32_t *start_state,
                        int32_t *done_state, int32_t *n_classes, uint64_t *content_hash) {
    if (!g) return WG_ERR_ARG;
    if (n_states) *n_states = g->n_states;
    if (start_state) *start_state = g->start;
    if (done_state) *done_state = g->done;
    if (n_classes) *n_classes = g->n_classes;
    if (content_hash) *content_hash = g->hash;
    return WG_OK;
}

int32_t wg_grammar_forced_token(const wg_grammar *g, int32_t state, int32_t *token,
                                int32_t *next_state) {
    if (!g || state < 0 || state >= g->n_states || g->forced_tok.empty()) return 0;
    if (g->forced_tok[state] < 0) return 0;
    if (token) *token = g->forced_tok[state];
    if (next_state) *next_state = g->forced_next[state];
    return 1;
}

int32_t wg_grammar_step(const wg_grammar *g, int32_t state, int32_t symbol) {
    if (!g || state < 0 || state >= g->n_states || symbol < 0 || symbol >= WG_N_SYMBOLS) return 0;
    const int c = symbol == WG_SYM_EOS ? g->eos_class : g->byte_class[symbol];
    return g->table[(size_t)state * g->n_classes + c];
}

// ---- context ------------------------------------------------------------------------

int32_t wg_ctx_create(const wg_vocab *vocab, int32_t cache_capacity, int32_t max_batch,
                      wg_ctx **out) {
    return wg_ctx_create_ex(vocab, cache_capacity, max_batch, WG_CACHE_DENSE, 0, out);
}

int32_t wg_ctx_create_ex(const wg_vocab *vocab, int32_t cache_capacity, int32_t max_batch,
                         int32_t cache_mode, size_t arena_bytes, wg_ctx **out) {
    if (!out) return WG_ERR_ARG;
    *out = nullptr;
    if (!vocab || cache_capacity < 0 || max_batch <= 0 || max_batch > WG_MAX_ROWS ||
        cache_capacity > (1 << 28))
        return WG_ERR_ARG;
    if (cache_mode != WG_CACHE_DENSE && cache_mode != WG_CACHE_COMPACT) return WG_ERR_ARG;
    const bool compact = cache_mode == WG_CACHE_COMPACT && cache_capacity > 0;
    wg_ctx *c = new (std::nothrow) wg_ctx();
    if (!c) return WG_ERR_ARG;
    c->vocab = vocab;
    c->max_batch = max_batch;
    memset(c->after_slot, 0xFF, sizeof(c->after_slot));
    CtxDev &d = c->dev;
    d.capacity = cache_capacity;
    d.pool_stride = ((int64_t)vocab->dev.W + 31) / 32 * 32;  // rows start on 128-byte lines
    d.hash_size = 0;
    if (cache_capacity > 0) {
        int32_t h = 64;
        while (h < 2 * cache_capacity) h <<= 1;
        d.hash_size = h;
    }
    int32_t rc = WG_OK;
    auto take = [&](auto **p, size_t n) {
        if (rc != WG_OK) return;
        rc = dev_alloc(p, n);
        if (rc == WG_OK) c->owned.push_back((void *)*p);
    };
    take(&d.keys, (size_t)d.hash_size);
    take(&d.vals, (size_t)d.hash_size);
    if (compact) {
        d.compact = 1;
        d.hdr_stride = (vocab->dev.W + 31) / 32;
        // at least one mask with every word stored; word offsets must fit in 31 bits
        size_t words = arena_bytes ? arena_bytes / sizeof(uint32_t)
                                   : (size_t)d.capacity * (size_t)d.pool_stride / 4;
        if (words < (size_t)d.pool_stride) words = (size_t)d.pool_stride;
        if (words > 0x7FFFFFFFull) words = 0x7FFFFFFFull;
        d.arena_words = (long long)words;
        take(&d.arena, (size_t)d.arena_words);
        take(&d.arena_top, 1);
        take(&d.ent_hdr, (size_t)d.capacity * (size_t)d.hdr_stride);
        take(&d.ent_fail, (size_t)d.capacity);
        take(&d.ent_stage, (size_t)d.capacity);
        take(&d.stage, (size_t)max_batch * (size_t)d.pool_stride);
        take(&d.bl_row, (size_t)max_batch);
    } else {
        take(&d.pool, (size_t)d.capacity * (size_t)d.pool_stride);
    }
    take(&d.n_slots, 1);
    take(&d.free_rows, (size_t)d.capacity);
    take(&d.n_free, 1);
    take(&c->d_counts, 1);
    take(&d.ent, (size_t)max_batch);
    take(&d.slot, (size_t)max_batch);
    take(&d.bl_gid, (size_t)max_batch);
    take(&d.bl_sid, (size_t)max_batch);
    take(&d.bl_dst, (size_t)max_batch);
    take(&d.bl_count, 1);
    take(&d.build_next, 2);
    take(&d.argkey, (size_t)max_batch);
    take(&d.stats, (size_t)ST_COUNT);
    take(&d.row_done, (size_t)max_batch);
    take(&c->d_stage_gid, (size_t)max_batch);
    take(&c->d_stage_sid, (size_t)max_batch);
    c->grammar_cap = 64;
    take(&c->d_grammars, (size_t)c->grammar_cap);
    if (rc == WG_OK) {
        d.build_done = d.build_next + 1;
        d.grammars = c->d_grammars;
        d.n_grammars = 0;
        if (cudaMemset(d.keys, 0, sizeof(unsigned long long) * (size_t)(d.hash_size ? d.hash_size : 1)) != cudaSuccess ||
            cudaMemset(d.vals, 0xFF, sizeof(int32_t) * (size_t)(d.hash_size ? d.hash_size : 1)) != cudaSuccess ||
            cudaMemset(d.n_slots, 0, sizeof(int32_t)) != cudaSuccess ||
            cudaMemset(d.n_free, 0, sizeof(int32_t)) != cudaSuccess ||
            cudaMemset(d.bl_count, 0, sizeof(int32_t)) != cudaSuccess ||
            cudaMemset(d.build_next, 0, 2 * sizeof(int32_t)) != cudaSuccess ||
            cudaMemset(d.argkey, 0, sizeof(unsigned long long) * (size_t)max_batch) != cudaSuccess ||
            cudaMemset(d.stats, 0, sizeof(unsigned long long) * ST_COUNT) != cudaSuccess ||
            cudaMemset(d.row_done, 0, sizeof(int32_t) * (size_t)max_batch) != cudaSuccess)
            rc = WG_ERR_CUDA;
        if (compact && rc == WG_OK &&
            (cudaMemset(d.arena_top, 0, sizeof(unsigned long long)) != cudaSuccess ||
             cudaMemset(d.ent_fail, 0, sizeof(int32_t) * (size_t)d.capacity) != cudaSuccess))
            rc = WG_ERR_CUDA;
    }
    if (rc != WG_OK) {
        wg_ctx_free(c);
        return rc;
    }
    *out = c;
    return WG_OK;
}

void wg_ctx_free(wg_ctx *c) {
    if (!c) return;
    cudaDeviceSynchronize();
    for (void *p : c->owned) cudaFree(p);
    cudaFree(c->d_after_masks);
    cudaFree(c->d_after_slot);
    cudaFree(c->d_leave_bits);
    for (ClassMappedRecords &r : c->class_records) cudaFree(r.d_rec);
    for (cudaEvent_t e : c->events) cudaEventDestroy(e);
    for (GrammarSlot &s : c->slots) {
        cudaFree(s.d_table);
        cudaFree(s.d_cls);
        cudaFree(s.d_first_ok);
        cudaFree(s.d_leaves);
        cudaFree(s.d_forced);
        cudaFree(s.d_leave1);
        cudaFree(s.d_leave_fold);
    }
    delete c;
}

int32_t wg_ctx_add_grammar(wg_ctx *c, const wg_grammar *g, int32_t *grammar_id) {
    NvtxRange nvtx_range("wg_ctx_add_grammar");
    if (!c || !g || !grammar_id) return WG_ERR_ARG;
    std::lock_guard<std::mutex> lock(c->mu);
    for (size_t i = 0; i < c->slots.size(); ++i) {
        if (c->slots[i].same_as(*g)) {
            *grammar_id = (int32_t)i;
            return WG_OK;
        }
    }
    bool id_waiting = false;  // the id of a removed grammar can be used again
    for (const GrammarSlot &sl : c->slots) id_waiting = id_waiting || sl.removed;
    if (c->slots.size() >= 65535 && !id_waiting) return WG_ERR_CAPACITY;
    // the kernels index table cells with 32 bits
    if ((uint64_t)g->n_states * (uint64_t)g->n_classes >= (1ull << 32)) return WG_ERR_CAPACITY;
    const bool wide = g->n_states > 65535;
    GrammarSlot slot{g->hash, g->table, g->forced_tok, g->forced_next, g->n_states, g->n_classes,
                     nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr,
                     {}, g->start, g->done, g->eos_class};
    memcpy(slot.byte_class, g->byte_class, 256);
    struct Guard {  // frees the uploads again if any later step fails
        GrammarSlot *s;
        ~Guard() {
            if (!s) return;
            cudaFree(s->d_table); cudaFree(s->d_cls); cudaFree(s->d_first_ok);
            cudaFree(s->d_leaves); cudaFree(s->d_forced); cudaFree(s->d_leave1); cudaFree(s->d_leave_fold);
        }
    } guard{&slot};
    if (!g->forced_tok.empty()) {
        std::vector<int2> forced(g->n_states);
        for (int32_t st = 0; st < g->n_states; ++st) forced[st] = make_int2(g->forced_tok[st], g->forced_next[st]);
        WG_CUDA(cudaMalloc(&slot.d_forced, forced.size() * sizeof(int2)));
        WG_CUDA(cudaMemcpy(slot.d_forced, forced.data(), forced.size() * sizeof(int2),
                           cudaMemcpyHostToDevice));
    }
    const size_t n = g->table.size();
    if (wide) {
        WG_CUDA(cudaMalloc(&slot.d_table, n * sizeof(uint32_t)));
        WG_CUDA(cudaMemcpy(slot.d_table, g->table.data(), n * sizeof(uint32_t), cudaMemcpyHostToDevice));
    } else {
        std::vector<uint16_t> narrow(n);
        for (size_t i = 0; i < n; ++i) narrow[i] = (uint16_t)g->table[i];
        WG_CUDA(cudaMalloc(&slot.d_table, n * sizeof(uint16_t)));
        WG_CUDA(cudaMemcpy(slot.d_table, narrow.data(), n * sizeof(uint16_t), cudaMemcpyHostToDevice));
    }
    WG_CUDA(cudaMalloc(&slot.d_cls, 256));
    WG_CUDA(cudaMemcpy(slot.d_cls, g->byte_class, 256, cudaMemcpyHostToDevice));
    // per state: the bytes that keep it alive, and (folded mod 64) the bytes that leave it
    {
        const int32_t S = g->n_states, C = g->n_classes;
        WG_CUDA(cudaMalloc(&slot.d_first_ok, (size_t)S * 8 * sizeof(uint32_t)));
        WG_CUDA(cudaMalloc(&slot.d_leaves, (size_t)S * sizeof(unsigned long long)));
        WG_CUDA(cudaMalloc(&slot.d_leave1, (size_t)S * sizeof(int16_t)));
        WG_CUDA(cudaMalloc(&slot.d_leave_fold, (size_t)S * sizeof(unsigned long long)));
        if (!c->d_leave_bits) WG_CUDA(cudaMalloc((void **)&c->d_leave_bits, 8 * sizeof(uint32_t)));
        WG_CUDA(cudaMemsetAsync(c->d_leave_bits, 0, 8 * sizeof(uint32_t), cudaStreamLegacy));
        const uint8_t *d_cls = static_cast<const uint8_t *>(slot.d_cls);
        uint32_t *d_ok = static_cast<uint32_t *>(slot.d_first_ok);
        int16_t *d_l1 = static_cast<int16_t *>(slot.d_leave1);
        unsigned long long *d_lf = static_cast<unsigned long long *>(slot.d_leave_fold);
        if (wide) {
            const uint32_t *tab = static_cast<const uint32_t *>(slot.d_table);
            grammar_state_info_kernel<uint32_t><<<(unsigned)S, 256, 0, cudaStreamLegacy>>>(
                tab, d_cls, S, C, d_ok, static_cast<unsigned long long *>(slot.d_leaves), d_l1);
            WG_LAUNCHED();
            leave_info_kernel<uint32_t><<<(unsigned)((S + 255) / 256), 256, 0, cudaStreamLegacy>>>(
                tab, d_cls, d_ok, d_l1, S, C, d_lf, c->d_leave_bits);
        } else {
            const uint16_t *tab = static_cast<const uint16_t *>(slot.d_table);
            grammar_state_info_kernel<uint16_t><<<(unsigned)S, 256, 0, cudaStreamLegacy>>>(
                tab, d_cls, S, C, d_ok, static_cast<unsigned long long *>(slot.d_leaves), d_l1);
            WG_LAUNCHED();
            leave_info_kernel<uint16_t><<<(unsigned)((S + 255) / 256), 256, 0, cudaStreamLegacy>>>(
                tab, d_cls, d_ok, d_l1, S, C, d_lf, c->d_leave_bits);
        }
        WG_LAUNCHED();
        // the bytes that close a free-text slot of this grammar get their vocabulary masks now
        uint32_t leave_bits[8];
        WG_CUDA(cudaMemcpy(leave_bits, c->d_leave_bits, sizeof(leave_bits), cudaMemcpyDeviceToHost));
        const VocabDev &v = c->vocab->dev;
        const size_t slot_words = (size_t)AFTER_ROWS * (size_t)v.W;
        bool table_changed = false;
        for (int b = 0; b < 256; ++b) {
            if (!((leave_bits[b >> 5] >> (b & 31)) & 1u) || c->after_slot[b] >= 0) continue;
            if (c->n_after >= AFTER_SLOTS) break;  // the rest goes without (results are the same)
            if (!c->d_after_masks) {
                WG_CUDA(cudaMalloc((void **)&c->d_after_masks, AFTER_SLOTS * slot_words * sizeof(uint32_t)));
                WG_CUDA(cudaMalloc((void **)&c->d_after_slot, 256));
            }
            uint32_t *rows = c->d_after_masks + (size_t)c->n_after * slot_words;
            WG_CUDA(cudaMemsetAsync(rows, 0, slot_words * sizeof(uint32_t), cudaStreamLegacy));
            after_masks_kernel<<<(unsigned)((v.W * 32 + 255) / 256), 256, 0, cudaStreamLegacy>>>(v, b, rows);
            WG_LAUNCHED();
            c->after_slot[b] = (int8_t)c->n_after++;
            table_changed = true;
        }
        if (table_changed) {
            WG_CUDA(cudaMemcpyAsync(c->d_after_slot, c->after_slot, 256, cudaMemcpyHostToDevice,
                                    cudaStreamLegacy));
            c->dev.after_masks = c->d_after_masks;
            c->dev.after_slot = c->d_after_slot;
        }
    }
    // the vocabulary's records with bytes replaced by this grammar's classes (shared between
    // grammars whose class maps are equal)
    const void *d_rec_class = nullptr;
    for (ClassMappedRecords &r : c->class_records)
        if (r.d_rec && memcmp(r.byte_class, g->byte_class, 256) == 0) {
            d_rec_class = r.d_rec;
            ++r.users;
            break;
        }
    if (!d_rec_class) {
        const int V = c->vocab->dev.V;
        ClassMappedRecords r;
        memcpy(r.byte_class, g->byte_class, 256);
        r.d_rec = nullptr;
        r.users = 1;
        WG_CUDA(cudaMalloc(&r.d_rec, (size_t)V * WG_REC_BYTES));
        map_records_kernel<<<(unsigned)((V + 255) / 256), 256, 0, cudaStreamLegacy>>>(
            c->vocab->dev.rec, static_cast<const uint8_t *>(slot.d_cls), static_cast<uint4 *>(r.d_rec), V);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (cudaGetLastError() != cudaSuccess) {
            cudaFree(r.d_rec);
            return WG_ERR_CUDA;
        }
        c->class_records.push_back(r);
        d_rec_class = r.d_rec;
    }
    // both kernels have finished before the grammar is used, on whatever stream that will be
    WG_CUDA(cudaStreamSynchronize(cudaStreamLegacy));
    GrammarDev gd{slot.d_table, static_cast<const uint8_t *>(slot.d_cls),
                  static_cast<const uint32_t *>(slot.d_first_ok),
                  static_cast<const unsigned long long *>(slot.d_leaves),
                  static_cast<const int2 *>(slot.d_forced),
                  static_cast<const uint4 *>(d_rec_class),
                  static_cast<const int16_t *>(slot.d_leave1),
                  static_cast<const unsigned long long *>(slot.d_leave_fold), g->n_states,
                  g->n_classes, g->start, g->done, g->eos_class, wide ? 1 : 0};
    int32_t id = (int32_t)c->slots.size();
    for (size_t i = 0; i < c->slots.size(); ++i)  // the id of a removed grammar is used again
        if (c->slots[i].removed) { id = (int32_t)i; break; }
    if (id >= c->grammar_cap) {  // grow the registry; queued kernels still read the old one
        WG_CUDA(cudaDeviceSynchronize());
        const int32_t cap = c->grammar_cap * 2;
        GrammarDev *bigger = nullptr;
        WG_CUDA(cudaMalloc((void **)&bigger, sizeof(GrammarDev) * (size_t)cap));
        WG_CUDA(cudaMemcpy(bigger, c->grammars.data(), sizeof(GrammarDev) * c->grammars.size(),
                           cudaMemcpyHostToDevice));
        c->owned.push_back(bigger);  // the old array is freed with the context
        c->d_grammars = bigger;
        c->grammar_cap = cap;
        c->dev.grammars = bigger;
    }
    WG_CUDA(cudaMemcpy(c->d_grammars + id, &gd, sizeof(GrammarDev), cudaMemcpyHostToDevice));
    guard.s = nullptr;  // the context owns the uploads from here on
    if (id < (int32_t)c->slots.size()) {
        c->grammars[id] = gd;
        c->slots[id] = std::move(slot);
    } else {
        c->grammars.push_back(gd);
        c->slots.push_back(std::move(slot));
        c->dev.n_grammars = id + 1;
    }
    *grammar_id = id;
    return WG_OK;
}

int32_t wg_ctx_remove_grammar(wg_ctx *c, int32_t grammar_id) {
    NvtxRange nvtx_range("wg_ctx_remove_grammar");
    if (!c) return WG_ERR_ARG;
    std::lock_guard<std::mutex> lock(c->mu);
    if (grammar_id < 0 || grammar_id >= (int32_t)c->slots.size() || c->slots[grammar_id].removed)
        return WG_ERR_ARG;
    // every queued kernel may still read the grammar's tables and the cache
    WG_CUDA(cudaDeviceSynchronize());
    GrammarSlot &slot = c->slots[grammar_id];
    // 1. rows that still name the id get an all-zero mask and a bad-state count from now on
    GrammarDev none{};
    WG_CUDA(cudaMemcpy(c->d_grammars + grammar_id, &none, sizeof(GrammarDev), cudaMemcpyHostToDevice));
    c->grammars[grammar_id] = none;
    // 2. its cached masks stop matching and their pool rows are handed out again
    if (c->dev.hash_size > 0) {
        WG_CUDA(cudaMemset(c->d_counts, 0, sizeof(int32_t)));
        remove_grammar_entries_kernel<<<(c->dev.hash_size + 255) / 256, 256, 0, cudaStreamLegacy>>>(
            c->dev, grammar_id, c->d_counts);
        WG_LAUNCHED();
        int32_t dropped = 0;
        WG_CUDA(cudaMemcpy(&dropped, c->d_counts, sizeof(dropped), cudaMemcpyDeviceToHost));
        c->removed_keys += dropped;
        // 3. once a quarter of the table is held by removed entries it is rebuilt without them
        if (c->removed_keys * 4 > c->dev.hash_size) {
            unsigned long long *old_keys = nullptr;
            int32_t *old_vals = nullptr;
            const size_t n = (size_t)c->dev.hash_size;
            if (cudaMalloc((void **)&old_keys, n * sizeof(unsigned long long)) != cudaSuccess ||
                cudaMalloc((void **)&old_vals, n * sizeof(int32_t)) != cudaSuccess) {
                cudaFree(old_keys);
                cudaGetLastError();   // (the table stays as it is: longer probes, same results)
            } else {
                cudaMemcpy(old_keys, c->dev.keys, n * sizeof(unsigned long long), cudaMemcpyDeviceToDevice);
                cudaMemcpy(old_vals, c->dev.vals, n * sizeof(int32_t), cudaMemcpyDeviceToDevice);
                cudaMemset(c->dev.keys, 0, n * sizeof(unsigned long long));
                cudaMemset(c->dev.vals, 0xFF, n * sizeof(int32_t));
                rehash_kernel<<<(unsigned)((n + 255) / 256), 256, 0, cudaStreamLegacy>>>(c->dev, old_keys, old_vals);
                WG_LAUNCHED();
                const cudaError_t err = cudaDeviceSynchronize();
                cudaFree(old_keys);
                cudaFree(old_vals);
                if (err != cudaSuccess) return WG_ERR_CUDA;
                c->removed_keys = 0;
            }
        }
    }
    WG_CUDA(cudaDeviceSynchronize());
    // 4. the grammar's own device arrays
    cudaFree(slot.d_table); cudaFree(slot.d_cls); cudaFree(slot.d_first_ok); cudaFree(slot.d_leaves);
    cudaFree(slot.d_forced); cudaFree(slot.d_leave1); cudaFree(slot.d_leave_fold);
    slot.d_table = slot.d_cls = slot.d_first_ok = slot.d_leaves = nullptr;
    slot.d_forced = slot.d_leave1 = slot.d_leave_fold = nullptr;
    for (ClassMappedRecords &r : c->class_records)
        if (r.d_rec && memcmp(r.byte_class, slot.byte_class, 256) == 0 && --r.users == 0) {
            cudaFree(r.d_rec);
            r.d_rec = nullptr;
        }
    slot.table.clear(); slot.table.shrink_to_fit();
    slot.forced_tok.clear(); slot.forced_next.clear();
    slot.removed = true;
    return WG_OK;
}

int32_t wg_cache_clear(wg_ctx *c, void *stream) {
    if (!c) return WG_ERR_ARG;
    c->part_begin = c->part_end = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int n = c->dev.hash_size > 0 ? c->dev.hash_size : 1;
    cache_clear_kernel<<<(n + 255) / 256, 256, 0, st>>>(c->dev);
    WG_LAUNCHED();
    c->removed_keys = 0;
    return WG_OK;
}

int32_t wg_get_stats(wg_ctx *c, wg_stats *out, void *stream) {
    if (!c || !out) return WG_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned long long h[ST_COUNT];
    int32_t n_slots = 0, n_free = 0;
    unsigned long long arena_top = 0;
    WG_CUDA(cudaMemcpyAsync(h, c->dev.stats, sizeof(h), cudaMemcpyDeviceToHost, st));
    WG_CUDA(cudaMemcpyAsync(&n_slots, c->dev.n_slots, sizeof(n_slots), cudaMemcpyDeviceToHost, st));
    WG_CUDA(cudaMemcpyAsync(&n_free, c->dev.n_free, sizeof(n_free), cudaMemcpyDeviceToHost, st));
    if (c->dev.compact)
        WG_CUDA(cudaMemcpyAsync(&arena_top, c->dev.arena_top, sizeof(arena_top),
                                cudaMemcpyDeviceToHost, st));
    WG_CUDA(cudaStreamSynchronize(st));
    out->cache_hits = (int64_t)h[ST_HITS];
    out->cache_misses = (int64_t)h[ST_MISSES];
    out->masks_built = (int64_t)h[ST_BUILT];
    out->rows_uncached = (int64_t)h[ST_UNCACHED];
    out->tokens_rejected = (int64_t)h[ST_REJECTED];
    out->empty_masks = (int64_t)h[ST_EMPTY];
    out->bad_states = (int64_t)h[ST_BAD_STATE];
    n_slots -= n_free > 0 ? n_free : 0;  // rows that a removed grammar gave back hold nothing
    out->cache_entries = n_slots;
    if (arena_top > (unsigned long long)c->dev.arena_words) arena_top = (unsigned long long)c->dev.arena_words;
    out->cache_bytes = c->dev.compact
        ? (int64_t)(arena_top * sizeof(uint32_t)) + (int64_t)n_slots * c->dev.hdr_stride * (int64_t)sizeof(uint2)
        : (int64_t)n_slots * c->dev.pool_stride * (int64_t)sizeof(uint32_t);
    return WG_OK;
}

int32_t wg_reset_stats(wg_ctx *c, void *stream) {
    if (!c) return WG_ERR_ARG;
    WG_CUDA(cudaMemsetAsync(c->dev.stats, 0, sizeof(unsigned long long) * ST_COUNT,
                            static_cast<cudaStream_t>(stream)));
    return WG_OK;
}

}  // extern "C"

// ---- launch helpers -------------------------------------------------------------------
namespace {

int32_t launch_build(wg_ctx *c, const BuildWork &work, int max_entries, cudaStream_t st,
                     bool pdl = false) {
    const VocabDev &v = c->vocab->dev;
    // few masks: small chunks so that one mask still spreads over many blocks
    BuildWork w = work;
    w.chunk = max_entries <= 32 ? 2048 : BUILD_CHUNK_MAX;
    if (w.t_last == 0) { w.t_first = 0; w.t_last = v.W * 32; }  // the whole vocabulary
    const long long n_chunks = ((long long)(w.t_last - w.t_first) + w.chunk - 1) / w.chunk;
    long long items = (long long)max_entries * n_chunks;
    if (items >= (1LL << 31)) return WG_ERR_CAPACITY;  // the kernel numbers its items with 32 bits
    auto kernel = c->dev.compact ? build_masks_kernel<true> : build_masks_kernel<false>;
    if (c->count_build_work)
        kernel = c->dev.compact ? build_masks_kernel<true, true> : build_masks_kernel<false, true>;
    // One block per resident slot: the blocks stride over the items, so blocks that had to wait
    // for a slot would start their equal share late and stretch the launch.
    int uncached_per_sm = 0;  // the counting variant is asked every time (it is never timed)
    int &per_sm = c->count_build_work ? uncached_per_sm : c->build_blocks_per_sm;
    if (per_sm == 0) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, BUILD_THREADS, 0) != cudaSuccess || n < 1)
            n = 4;
        per_sm = n;
    }
    long long grid = (long long)sm_count() * per_sm;
    if (items < grid) grid = items;
    if (grid < 1) grid = 1;
    if (pdl)
        WG_CUDA(launch_pdl(kernel, dim3((unsigned)grid), dim3(BUILD_THREADS), st, v, c->dev, w));
    else
        kernel<<<(unsigned)grid, BUILD_THREADS, 0, st>>>(v, c->dev, w);
    WG_LAUNCHED();
    return WG_OK;
}

bool rows_aligned(const void *p, int64_t stride_elems, size_t elem) {
    return ((uintptr_t)p % 16 == 0) && ((stride_elems * (int64_t)elem) % 16 == 0);
}

// Grid of the apply kernels, (blocks per row, B), and the spans each block handles: every
// warp of a block takes 1, 2 or 4 spans of 1024 tokens; the smaller counts are used while the
// grid would otherwise hold fewer than about four waves of blocks (a short last wave costs).
dim3 apply_grid(ApplyArgs &a) {
    const int n_spans = (a.W + 31) / 32 - a.span_first;
    int per_warp = APPLY_SPANS_PER_WARP;
    while (per_warp > 1 &&
           (long long)a.B * ((n_spans + APPLY_WARPS * per_warp - 1) / (APPLY_WARPS * per_warp)) <
               16LL * sm_count())
        per_warp >>= 1;
    a.spans_per_block = APPLY_WARPS * per_warp;
    const int blocks_per_row = (n_spans + a.spans_per_block - 1) / a.spans_per_block;
    return dim3((unsigned)blocks_per_row, (unsigned)a.B);
}

template <typename E, bool ARGMAX, bool GATHER>
int32_t launch_apply_t(const ApplyArgs &a_in, const CtxDev &ctx, unsigned long long *argkey,
                       cudaStream_t st, bool pdl) {
    ApplyArgs a = a_in;
    dim3 grid = apply_grid(a);
    const bool aligned = rows_aligned(a.logits, a.row_stride, sizeof(E));
    if (pdl) {
        if (aligned)
            WG_CUDA(launch_pdl(apply_mask_kernel<E, ARGMAX, GATHER>, grid, dim3(APPLY_THREADS), st,
                               a, ctx, argkey));
        else
            WG_CUDA(launch_pdl(apply_mask_unaligned_kernel<E, ARGMAX, GATHER>, grid,
                               dim3(APPLY_THREADS), st, a, ctx, argkey));
    } else if (aligned) {
        apply_mask_kernel<E, ARGMAX, GATHER><<<grid, APPLY_THREADS, 0, st>>>(a, ctx, argkey);
    } else {
        apply_mask_unaligned_kernel<E, ARGMAX, GATHER><<<grid, APPLY_THREADS, 0, st>>>(a, ctx, argkey);
    }
    WG_LAUNCHED();
    return WG_OK;
}

template <bool ARGMAX, bool GATHER>
int32_t launch_apply(int32_t dtype, const ApplyArgs &a, const CtxDev &ctx,
                     unsigned long long *argkey, cudaStream_t st, bool pdl = false) {
    if (dtype == WG_DTYPE_BF16)
        return launch_apply_t<uint16_t, ARGMAX, GATHER>(a, ctx, argkey, st, pdl);
    return launch_apply_t<uint32_t, ARGMAX, GATHER>(a, ctx, argkey, st, pdl);
}

bool batch_ok(const wg_ctx *c, int32_t B) { return c && B >= 1 && B <= c->max_batch; }

// wg_decode_step over at most this many rows is one kernel launch (measured on the JSON workload:
// 12.3 against 14.3 us per step at 64 rows; at 128 rows with half of them missing the cache the
// separate kernels win, 52 against 63 us)
constexpr int SMALL_STEP_ROWS = 64;

}  // namespace

extern "C" {

// ---- decode path ----------------------------------------------------------------------

int32_t wg_mask_cache_lookup(wg_ctx *c, const int32_t *gid, const int32_t *sid, int32_t B,
                             int32_t *slot, void *stream) {
    NvtxRange nvtx_range("wg_mask_cache_lookup");
    if (!batch_ok(c, B) || !gid || !sid || !slot) return WG_ERR_ARG;
    cache_lookup_kernel<<<(B + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        c->dev, gid, sid, B, slot);
    WG_LAUNCHED();
    return WG_OK;
}

int32_t wg_build_masks(wg_ctx *c, const int32_t *gid, const int32_t *sid, int32_t B,
                       uint32_t *bitmask, int64_t row_stride_words, uint32_t flags, void *stream) {
    NvtxRange nvtx_range("wg_build_masks");
    if (!batch_ok(c, B) || !gid || !sid || !bitmask) return WG_ERR_ARG;
    const int W = c->vocab->dev.W;
    if (row_stride_words < W || (flags & ~(uint32_t)WG_NO_CACHE)) return WG_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (flags & WG_NO_CACHE) {
        BuildWork work{gid, sid, nullptr, bitmask, row_stride_words, nullptr, B, 0, 0, 0};
        return launch_build(c, work, B, st);
    }
    if (c->part_end != 0) return WG_ERR_ARG;  // cached masks are partial: see wg_decode_step_shard
    cache_lookup_insert_kernel<<<1, 1024, 0, st>>>(c->dev, gid, sid, B, bitmask, row_stride_words);
    WG_LAUNCHED();
    BuildWork work{c->dev.bl_gid, c->dev.bl_sid, c->dev.bl_dst, nullptr, 0, c->dev.bl_count, 0, 0, 0, 0};
    int32_t rc = launch_build(c, work, B, st);
    if (rc != WG_OK) return rc;
    dim3 grid((unsigned)((W + 1023) / 1024), (unsigned)B);
    if (c->dev.compact)
        cache_gather_compact_kernel<<<grid, 256, 0, st>>>(c->dev, c->vocab->dev.V, W, bitmask,
                                                          row_stride_words);
    else
        cache_gather_kernel<<<grid, 256, 0, st>>>(c->dev, W, bitmask, row_stride_words);
    WG_LAUNCHED();
    return WG_OK;
}

size_t wg_apply_workspace_bytes(int32_t B) { return B > 0 ? sizeof(unsigned long long) * (size_t)B : 0; }

int32_t wg_apply_mask(void *logits, int32_t dtype, int64_t row_stride_elems,
                      const uint32_t *bitmask, int64_t mask_stride_words, int32_t B, int32_t V,
                      int32_t *argmax_out, void *workspace, void *stream) {
    NvtxRange nvtx_range("wg_apply_mask");
    if (!logits || !bitmask || B < 1 || B > WG_MAX_ROWS || V < 1) return WG_ERR_ARG;
    if (dtype != WG_DTYPE_BF16 && dtype != WG_DTYPE_FP32) return WG_ERR_ARG;
    const int W = (V + 31) / 32;
    if (row_stride_elems < V || mask_stride_words < W) return WG_ERR_ARG;
    if (argmax_out && (!workspace || (uintptr_t)workspace % 8 != 0)) return WG_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ApplyArgs a{logits, row_stride_elems, bitmask, nullptr, mask_stride_words, B, V, W, 0, 0};
    CtxDev none{};
    if (!argmax_out) return launch_apply<false, false>(dtype, a, none, nullptr, st);
    unsigned long long *keys = static_cast<unsigned long long *>(workspace);
    WG_CUDA(cudaMemsetAsync(keys, 0, sizeof(unsigned long long) * (size_t)B, st));
    int32_t rc = launch_apply<true, false>(dtype, a, none, keys, st);
    if (rc != WG_OK) return rc;
    argmax_finish_kernel<<<(B + 127) / 128, 128, 0, st>>>(keys, B, argmax_out);
    WG_LAUNCHED();
    return WG_OK;
}

}  // extern "C"

// ---- the entry point that allocates nothing ----------------------------------------------
// Scratch of wg_apply_mask_noalloc: the packed per-row maxima.  The array lives in the
// library image, so each GPU that loads the library carries these 32 KB until exit.  In HOST
// code the name below is only a handle for the runtime, never a device address; the address
// a kernel may use comes from cudaGetSymbolAddress, queried once per device.
static __device__ __align__(256) unsigned long long g_noalloc_argkeys[WG_NOALLOC_MAX_ROWS];

namespace {
constexpr int MAX_DEVICES = 64;
std::mutex g_noalloc_mu;
unsigned long long *g_noalloc_ptr[MAX_DEVICES] = {};

// Device address of the scratch array on the CURRENT device (looked up on first use).
int32_t noalloc_scratch(unsigned long long **out) {
    int dev = -1;
    WG_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return WG_ERR_ARG;
    std::lock_guard<std::mutex> lock(g_noalloc_mu);
    if (!g_noalloc_ptr[dev]) {
        void *p = nullptr;
        WG_CUDA(cudaGetSymbolAddress(&p, g_noalloc_argkeys));
        g_noalloc_ptr[dev] = static_cast<unsigned long long *>(p);
    }
    *out = g_noalloc_ptr[dev];
    return WG_OK;
}
}  // namespace

extern "C" {

int32_t wg_apply_mask_noalloc(void *logits, int32_t dtype, int64_t row_stride_elems,
                              const uint32_t *bitmask, int64_t mask_stride_words, int32_t B,
                              int32_t V, int32_t *argmax_out, void *stream) {
    if (!logits || !bitmask || !argmax_out || B < 1 || V < 1) return WG_ERR_ARG;
    if (dtype != WG_DTYPE_BF16 && dtype != WG_DTYPE_FP32) return WG_ERR_ARG;
    if (B > WG_NOALLOC_MAX_ROWS) return WG_ERR_CAPACITY;  // the fixed scratch holds no more rows
    const int W = (V + 31) / 32;
    if (row_stride_elems < V || mask_stride_words < W) return WG_ERR_ARG;
    unsigned long long *keys = nullptr;
    int32_t rc = noalloc_scratch(&keys);
    if (rc != WG_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array still holds the previous call's maxima: the rows in use must start at zero
    WG_CUDA(cudaMemsetAsync(keys, 0, sizeof(unsigned long long) * (size_t)B, st));
    ApplyArgs a{logits, row_stride_elems, bitmask, nullptr, mask_stride_words, B, V, W, 0, 0};
    CtxDev none{};
    rc = launch_apply<true, false>(dtype, a, none, keys, st);
    if (rc != WG_OK) return rc;
    argmax_finish_kernel<<<(B + 127) / 128, 128, 0, st>>>(keys, B, argmax_out);
    WG_LAUNCHED();
    return WG_OK;
}

int32_t wg_advance(wg_ctx *c, const int32_t *gid, int32_t *sid, const int32_t *token, int32_t B,
                   int32_t *status, uint32_t flags, void *stream) {
    NvtxRange nvtx_range("wg_advance");
    if (!batch_ok(c, B) || !gid || !sid || !token) return WG_ERR_ARG;
    if (flags & ~(uint32_t)WG_RESTART_ON_DONE) return WG_ERR_ARG;
    advance_kernel<<<(B + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        c->vocab->dev, c->dev, gid, sid, token, nullptr, B, status, flags, 0,
        (const long long *)nullptr);
    WG_LAUNCHED();
    return WG_OK;
}

}  // extern "C"

namespace {
// One decode step over the tokens [v_begin, v_end) of the vocabulary.  `logits` holds those
// tokens only (element 0 of a row is token v_begin).  With best_keys the step ends by handing
// the packed maxima to the caller instead of advancing the states.
int32_t decode_step_impl(wg_ctx *c, const int32_t *gid, int32_t *sid, int32_t B, void *logits,
                         int32_t dtype, int64_t row_stride_elems, uint32_t *bitmask,
                         int64_t mask_stride_words, int32_t v_begin, int32_t v_end,
                         int32_t *token_out, long long *best_keys, int32_t *status, uint32_t flags,
                         cudaStream_t st) {
    const VocabDev &v = c->vocab->dev;
    const bool no_cache = (flags & WG_NO_CACHE) != 0;
    const bool whole = v_begin == 0 && v_end == v.V;
    if (!no_cache) {
        // cached masks hold the words of one token range only once a partial step has run
        if (c->part_end != 0 && (c->part_begin != v_begin || c->part_end != v_end)) return WG_ERR_ARG;
        if (!whole) { c->part_begin = v_begin; c->part_end = v_end; }
    }
    const size_t esize = dtype == WG_DTYPE_BF16 ? 2 : 4;
    // token t of the vocabulary is element t of the (virtual) row that starts v_begin earlier
    void *row0 = static_cast<char *>(logits) - (size_t)v_begin * esize;
    const int W_end = (v_end + 31) / 32;
    ApplyArgs a{row0, row_stride_elems, bitmask, bitmask, mask_stride_words, B, v_end, W_end, 0,
                v_begin / 1024};
    const int32_t t_last = v_end == v.V ? v.W * 32 : v_end;
    // Without token_out and best_keys the step only masks: no argmax, no advance (the caller
    // samples and calls wg_advance).
    const bool mask_only = !token_out && !best_keys;
    if (whole && !best_keys && !mask_only && B <= SMALL_STEP_ROWS &&
        rows_aligned(logits, row_stride_elems, esize)) {
        // A handful of rows: the whole step in one launch (see decode_step_small_kernel).
        int32_t rc;
        if ((rc = timing_mark(c, 0, st)) != WG_OK) return rc;
        if ((rc = timing_mark(c, 1, st)) != WG_OK) return rc;
        if ((rc = timing_mark(c, 2, st)) != WG_OK) return rc;
        const dim3 grid = apply_grid(a);
        const SmallStepArgs ss{gid, sid, token_out, status, (uint32_t)(flags & WG_RESTART_ON_DONE),
                               no_cache ? 0 : 1};
        if (dtype == WG_DTYPE_BF16)
            WG_CUDA(launch_pdl(decode_step_small_kernel<uint16_t>, grid, dim3(APPLY_THREADS), st, a,
                               c->dev, v, ss));
        else
            WG_CUDA(launch_pdl(decode_step_small_kernel<uint32_t>, grid, dim3(APPLY_THREADS), st, a,
                               c->dev, v, ss));
        WG_LAUNCHED();
        return timing_mark(c, 3, st);
    }
    // Every kernel of the step is launched with programmatic stream serialization and starts
    // with griddepcontrol.wait, so launch latency and block scheduling of a kernel overlap the
    // tail of the one before it (also across consecutive steps on one stream).
    int32_t rc;
    if ((rc = timing_mark(c, 0, st)) != WG_OK) return rc;
    if (no_cache) {
        // rows have no pool row; the packed maxima were left at zero by the last advance
        WG_CUDA(launch_pdl(reset_rows_kernel, dim3((B + 255) / 256), dim3(256), st, c->dev, B));
        WG_LAUNCHED();
        BuildWork work{gid, sid, nullptr, bitmask, mask_stride_words, nullptr, B, 0, v_begin, t_last};
        rc = launch_build(c, work, B, st, true);
    } else {
        WG_CUDA(launch_pdl(cache_lookup_insert_kernel, dim3(1), dim3(1024), st, c->dev, gid, sid, B,
                           bitmask, mask_stride_words));
        WG_LAUNCHED();
        BuildWork work{c->dev.bl_gid, c->dev.bl_sid, c->dev.bl_dst, nullptr, 0, c->dev.bl_count, 0, 0,
                       v_begin, t_last};
        rc = launch_build(c, work, B, st, true);
    }
    if (rc != WG_OK) return rc;
    if ((rc = timing_mark(c, 1, st)) != WG_OK) return rc;
    if ((rc = timing_mark(c, 2, st)) != WG_OK) return rc;
    if (mask_only)
        rc = no_cache ? launch_apply<false, false>(dtype, a, c->dev, nullptr, st, true)
                      : launch_apply<false, true>(dtype, a, c->dev, nullptr, st, true);
    else
        rc = no_cache ? launch_apply<true, false>(dtype, a, c->dev, c->dev.argkey, st, true)
                      : launch_apply<true, true>(dtype, a, c->dev, c->dev.argkey, st, true);
    if (rc != WG_OK) return rc;
    if ((rc = timing_mark(c, 3, st)) != WG_OK) return rc;
    if (mask_only) return WG_OK;
    if (best_keys) {
        WG_CUDA(launch_pdl(export_keys_kernel, dim3((B + 127) / 128), dim3(128), st, c->dev,
                           best_keys, B));
        WG_LAUNCHED();
        return WG_OK;
    }
    WG_CUDA(launch_pdl(advance_kernel, dim3((B + 127) / 128), dim3(128), st, v, c->dev, gid, sid,
                       (const int32_t *)nullptr, token_out, B, status,
                       (uint32_t)(flags & WG_RESTART_ON_DONE), 1, (const long long *)nullptr));
    WG_LAUNCHED();
    return WG_OK;
}
}  // namespace

extern "C" {

int32_t wg_decode_step(wg_ctx *c, const int32_t *gid, int32_t *sid, int32_t B, void *logits,
                       int32_t dtype, int64_t row_stride_elems, uint32_t *bitmask,
                       int64_t mask_stride_words, int32_t *token_out, int32_t *status,
                       uint32_t flags, void *stream) {
    NvtxRange nvtx_range("wg_decode_step");
    if (!batch_ok(c, B) || !gid || !sid || !logits || !bitmask) return WG_ERR_ARG;
    if (dtype != WG_DTYPE_BF16 && dtype != WG_DTYPE_FP32) return WG_ERR_ARG;
    if (flags & ~(uint32_t)(WG_NO_CACHE | WG_RESTART_ON_DONE)) return WG_ERR_ARG;
    if (!token_out && (status || (flags & WG_RESTART_ON_DONE))) return WG_ERR_ARG;  // nothing advances
    const VocabDev &v = c->vocab->dev;
    if (row_stride_elems < v.V || mask_stride_words < v.W) return WG_ERR_ARG;
    return decode_step_impl(c, gid, sid, B, logits, dtype, row_stride_elems, bitmask,
                            mask_stride_words, 0, v.V, token_out, nullptr, status, flags,
                            static_cast<cudaStream_t>(stream));
}

int32_t wg_decode_step_shard(wg_ctx *c, const int32_t *gid, const int32_t *sid, int32_t B,
                             void *logits_shard, int32_t dtype, int64_t row_stride_elems,
                             uint32_t *bitmask, int64_t mask_stride_words, int32_t v_begin,
                             int32_t v_end, int64_t *best_keys, uint32_t flags, void *stream) {
    NvtxRange nvtx_range("wg_decode_step_shard");
    if (!batch_ok(c, B) || !gid || !sid || !logits_shard || !bitmask || !best_keys) return WG_ERR_ARG;
    if (dtype != WG_DTYPE_BF16 && dtype != WG_DTYPE_FP32) return WG_ERR_ARG;
    if (flags & ~(uint32_t)WG_NO_CACHE) return WG_ERR_ARG;
    const VocabDev &v = c->vocab->dev;
    if (v_begin < 0 || v_begin >= v_end || v_end > v.V || v_begin % WG_SHARD_ALIGN != 0 ||
        (v_end != v.V && v_end % WG_SHARD_ALIGN != 0))
        return WG_ERR_ARG;
    if (row_stride_elems < v_end - v_begin || mask_stride_words < v.W) return WG_ERR_ARG;
    static_assert(sizeof(long long) == sizeof(int64_t), "packed maxima are 64-bit");
    return decode_step_impl(c, gid, const_cast<int32_t *>(sid), B, logits_shard, dtype,
                            row_stride_elems, bitmask, mask_stride_words, v_begin, v_end, nullptr,
                            reinterpret_cast<long long *>(best_keys), nullptr, flags,
                            static_cast<cudaStream_t>(stream));
}

int32_t wg_advance_keys(wg_ctx *c, const int32_t *gid, int32_t *sid, const int64_t *best_keys,
                        int32_t B, int32_t *token_out, int32_t *status, uint32_t flags,
                        void *stream) {
    NvtxRange nvtx_range("wg_advance_keys");
    if (!batch_ok(c, B) || !gid || !sid || !best_keys || !token_out) return WG_ERR_ARG;
    if (flags & ~(uint32_t)WG_RESTART_ON_DONE) return WG_ERR_ARG;
    advance_kernel<<<(B + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        c->vocab->dev, c->dev, gid, sid, nullptr, token_out, B, status, flags, 2,
        reinterpret_cast<const long long *>(best_keys));
    WG_LAUNCHED();
    return WG_OK;
}

}  // extern "C"

struct wg_step_graph {
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    int64_t kernels = 0;  // kernel launches one replay stands for
};

extern "C" {

int32_t wg_step_graph_create(wg_ctx *c, const int32_t *gid, int32_t *sid, int32_t B, void *logits,
                             int32_t dtype, int64_t row_stride_elems, uint32_t *bitmask,
                             int64_t mask_stride_words, int32_t *token_out, int32_t *status,
                             uint32_t flags, wg_step_graph **out) {
    if (!out) return WG_ERR_ARG;
    *out = nullptr;
    if (!c) return WG_ERR_ARG;
    wg_step_graph *g = new (std::nothrow) wg_step_graph();
    if (!g) return WG_ERR_ARG;
    cudaStream_t cap = nullptr;
    int32_t rc = WG_OK;
    if (cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking) != cudaSuccess) rc = WG_ERR_CUDA;
    const bool timing = c->timing;
    c->timing = false;  // event records do not belong in the recorded step
    if (rc == WG_OK && cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal) != cudaSuccess)
        rc = WG_ERR_CUDA;
    if (rc == WG_OK) {
        const int64_t before = g_launches.load(std::memory_order_relaxed);
        rc = wg_decode_step(c, gid, sid, B, logits, dtype, row_stride_elems, bitmask,
                            mask_stride_words, token_out, status, flags, cap);
        // the launches were recorded, not run: take them off the count of launches made
        g->kernels = g_launches.load(std::memory_order_relaxed) - before;
        g_launches.fetch_sub(g->kernels, std::memory_order_relaxed);
        cudaGraph_t graph = nullptr;
        const cudaError_t e = cudaStreamEndCapture(cap, &graph);  // always end the capture
        if (rc == WG_OK && e != cudaSuccess) { g_last_cuda_error = (int32_t)e; rc = WG_ERR_CUDA; }
        g->graph = graph;
    }
    c->timing = timing;
    if (rc == WG_OK) {
        const cudaError_t e = cudaGraphInstantiate(&g->exec, g->graph, 0);
        if (e != cudaSuccess) { g_last_cuda_error = (int32_t)e; rc = WG_ERR_CUDA; }
    }
    if (cap) cudaStreamDestroy(cap);
    if (rc != WG_OK) {
        wg_step_graph_free(g);
        return rc;
    }
    *out = g;
    return WG_OK;
}

int32_t wg_step_graph_launch(wg_step_graph *g, void *stream) {
    if (!g || !g->exec) return WG_ERR_ARG;
    WG_CUDA(cudaGraphLaunch(g->exec, static_cast<cudaStream_t>(stream)));
    g_launches.fetch_add(g->kernels, std::memory_order_relaxed);  // the kernels of one step
    return WG_OK;
}

void wg_step_graph_free(wg_step_graph *g) {
    if (!g) return;
    if (g->exec) cudaGraphExecDestroy(g->exec);
    if (g->graph) cudaGraphDestroy(g->graph);
    delete g;
}

int32_t wg_decode_step_host(wg_ctx *c, const int32_t *gid, int32_t *sid, int32_t B,
                            const void *logits_host, void *logits_dev, int32_t dtype,
                            int64_t row_stride_elems, uint32_t *bitmask,
                            int64_t mask_stride_words, int32_t *token_dev, int32_t *token_host,
                            int32_t *status, uint32_t flags, void *stream) {
    NvtxRange nvtx_range("wg_decode_step_host");
    if (!c || !logits_host || !logits_dev || !token_dev || !token_host) return WG_ERR_ARG;
    if (dtype != WG_DTYPE_BF16 && dtype != WG_DTYPE_FP32) return WG_ERR_ARG;
    if (!batch_ok(c, B) || row_stride_elems < c->vocab->dev.V) return WG_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t e = dtype == WG_DTYPE_BF16 ? 2 : 4;
    const size_t row_bytes = (size_t)c->vocab->dev.V * e;
    WG_CUDA(cudaMemcpy2DAsync(logits_dev, (size_t)row_stride_elems * e, logits_host, row_bytes,
                              row_bytes, (size_t)B, cudaMemcpyHostToDevice, st));
    int32_t rc = wg_decode_step(c, gid, sid, B, logits_dev, dtype, row_stride_elems, bitmask,
                                mask_stride_words, token_dev, status, flags, stream);
    if (rc != WG_OK) return rc;
    WG_CUDA(cudaMemcpyAsync(token_host, token_dev, sizeof(int32_t) * (size_t)B,
                            cudaMemcpyDeviceToHost, st));
    WG_CUDA(cudaStreamSynchronize(st));
    return WG_OK;
}

int32_t wg_ctx_count_build_work(wg_ctx *c, int32_t enable) {
    if (!c) return WG_ERR_ARG;
    c->count_build_work = enable != 0;
    return WG_OK;
}

int32_t wg_get_build_work(wg_ctx *c, int64_t *tokens_walked, int64_t *table_lookups,
                          int64_t *mask_words_read, void *stream) {
    if (!c) return WG_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned long long h[ST_COUNT];
    WG_CUDA(cudaMemcpyAsync(h, c->dev.stats, sizeof(h), cudaMemcpyDeviceToHost, st));
    WG_CUDA(cudaStreamSynchronize(st));
    if (tokens_walked) *tokens_walked = (int64_t)h[ST_QUEUED];
    if (table_lookups) *table_lookups = (int64_t)h[ST_WALKED];
    if (mask_words_read) *mask_words_read = (int64_t)h[ST_MASK_WORDS];
    return WG_OK;
}

int32_t wg_ctx_set_timing(wg_ctx *c, int32_t enable) {
    if (!c) return WG_ERR_ARG;
    c->timing = enable != 0;
    c->timed_steps = 0;
    return WG_OK;
}

int32_t wg_ctx_get_timing(wg_ctx *c, double *build_ms, double *apply_ms, int64_t *steps) {
    if (!c) return WG_ERR_ARG;
    double b = 0.0, a = 0.0;
    for (size_t i = 0; i < c->timed_steps; ++i) {
        float ms = 0.f;
        WG_CUDA(cudaEventSynchronize(c->events[4 * i + 3]));
        WG_CUDA(cudaEventElapsedTime(&ms, c->events[4 * i], c->events[4 * i + 1]));
        b += ms;
        WG_CUDA(cudaEventElapsedTime(&ms, c->events[4 * i + 2], c->events[4 * i + 3]));
        a += ms;
    }
    if (build_ms) *build_ms = b;
    if (apply_ms) *apply_ms = a;
    if (steps) *steps = (int64_t)c->timed_steps;
    c->timed_steps = 0;
    return WG_OK;
}

int32_t wg_cache_entry_read(wg_ctx *c, int32_t grammar_id, int32_t state, int32_t *kind,
                            int32_t *n_listed, int32_t *ids_host, int32_t ids_capacity,
                            int64_t *entry_bytes, void *stream) {
    if (!c || !c->dev.compact || ids_capacity < 0 || (ids_capacity > 0 && !ids_host)) return WG_ERR_ARG;
    if (c->part_end != 0) return WG_ERR_ARG;  // cached masks hold one vocabulary slice only
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const VocabDev &v = c->vocab->dev;
    if (kind) *kind = -1;
    if (n_listed) *n_listed = 0;
    if (entry_bytes) *entry_bytes = 0;
    // find the cache row with the device's own probe and let the device expand the entry into
    // a scratch row, exactly as a decode step reads it
    iota_states_kernel<<<1, 32, 0, st>>>(c->d_stage_gid, c->d_stage_sid, grammar_id, state, 1);
    WG_LAUNCHED();
    cache_lookup_kernel<<<1, 32, 0, st>>>(c->dev, c->d_stage_gid, c->d_stage_sid, 1, c->dev.slot);
    WG_LAUNCHED();
    int32_t row = -1;
    WG_CUDA(cudaMemcpyAsync(&row, c->dev.slot, sizeof(row), cudaMemcpyDeviceToHost, st));
    WG_CUDA(cudaStreamSynchronize(st));
    if (row < 0) return WG_OK;
    cache_gather_compact_kernel<<<dim3((unsigned)((v.W + 1023) / 1024), 1), 256, 0, st>>>(
        c->dev, v.V, v.W, c->dev.stage, c->dev.pool_stride);
    WG_LAUNCHED();
    std::vector<uint32_t> words((size_t)v.W);
    std::vector<uint2> hdr((size_t)c->dev.hdr_stride);
    WG_CUDA(cudaMemcpyAsync(words.data(), c->dev.stage, words.size() * sizeof(uint32_t),
                            cudaMemcpyDeviceToHost, st));
    WG_CUDA(cudaMemcpyAsync(hdr.data(), c->dev.ent_hdr + (size_t)row * c->dev.hdr_stride,
                            hdr.size() * sizeof(uint2), cudaMemcpyDeviceToHost, st));
    WG_CUDA(cudaStreamSynchronize(st));
    // the paper's rule for the mask as a whole: keep the side with fewer tokens
    int64_t allowed = 0;
    for (uint32_t w : words) allowed += __builtin_popcount(w);
    const int32_t k = 2 * allowed <= (int64_t)v.V ? WG_ENTRY_ALLOWS : WG_ENTRY_DENIES;
    int32_t written = 0, total = 0;
    for (int w = 0; w < v.W; ++w) {
        const int tail = v.V & 31;
        const uint32_t full = (w == v.W - 1 && tail) ? ((1u << tail) - 1u) : 0xFFFFFFFFu;
        uint32_t listed = (k == WG_ENTRY_ALLOWS ? words[w] : ~words[w]) & full;
        while (listed) {
            const int b = __builtin_ctz(listed);
            listed &= listed - 1;
            if (written < ids_capacity) ids_host[written++] = w * 32 + b;
            ++total;
        }
    }
    size_t stored = 0;
    for (const uint2 &h : hdr) stored += (size_t)__builtin_popcount(h.x);
    if (kind) *kind = k;
    if (n_listed) *n_listed = total;
    if (entry_bytes) *entry_bytes = (int64_t)(hdr.size() * sizeof(uint2) + stored * sizeof(uint32_t));
    return WG_OK;
}

int32_t wg_cache_prewarm(wg_ctx *c, int32_t grammar_id, void *stream) {
    NvtxRange nvtx_range("wg_cache_prewarm");
    if (!c || grammar_id < 0 || grammar_id >= (int32_t)c->slots.size()) return WG_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int32_t S = c->slots[grammar_id].n_states;
    wg_stats before{}, after{};
    int32_t rc = wg_get_stats(c, &before, stream);
    if (rc != WG_OK) return rc;
    for (int32_t first = 1; first < S; first += c->max_batch) {
        const int32_t n = (S - first < c->max_batch) ? S - first : c->max_batch;
        iota_states_kernel<<<(n + 255) / 256, 256, 0, st>>>(c->d_stage_gid, c->d_stage_sid,
                                                            grammar_id, first, n);
        WG_LAUNCHED();
        cache_lookup_insert_kernel<<<1, 1024, 0, st>>>(c->dev, c->d_stage_gid, c->d_stage_sid, n,
                                                       nullptr, 0);
        WG_LAUNCHED();
        BuildWork work{c->dev.bl_gid, c->dev.bl_sid, c->dev.bl_dst, nullptr, 0, c->dev.bl_count, 0, 0, 0, 0};
        rc = launch_build(c, work, n, st);
        if (rc != WG_OK) return rc;
        // a batch that found the pool (or the arena) full ends the prewarm: later batches would
        // only be looked up and dropped
        rc = wg_get_stats(c, &after, stream);
        if (rc != WG_OK) return rc;
        if (after.rows_uncached > before.rows_uncached) return WG_ERR_CAPACITY;
    }
    return WG_OK;
}

}  // extern "C"
