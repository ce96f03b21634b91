// C ABI of libunity: argument validation, workspace carving and the launch sequence of each call.
// All arithmetic of the path runs in the kernels of stream_kernels.cu and gemm_tcgen05.cu.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "internal.h"

using namespace unity;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct unity_ctx {
    int device;
    cudaStream_t stream;
    char* ws;
    size_t ws_bytes;
    int* d_status;        // device status word
    int* h_pinned;        // pinned host staging for the per-model counts and the status word
    int sm_count;
    EncodeTiledFn encode;
    long long launches;
    char err[512];
    // optional per-kernel-class timing (unity_set_profiling): pairs of events around each launch
    int profiling;
    std::vector<cudaEvent_t>* ev_pool;
    std::vector<int>* ev_class;     // class of the i-th recorded pair
    size_t ev_used;                 // events handed out since the last unity_get_profile
    int ctas[UNITY_PROF_CLASSES];   // per GEMM class: 1 = single CTA per tile, 2 = CTA pair per tile
    int l2_promotion;               // tensor-map L2 promotion: 0 none, 1 64 B, 2 128 B, 3 256 B
    int chunk_group[3];             // raster group of the recompute / dHidden / dW chunk GEMMs, in 128-row tiles
    int chunk_rows_mult, chunk_vocab_mult;   // gradient chunk = mult x 18944 rows / vocabulary entries
    int fwd_group;                  // row tiles (128 rows) per round of the forward kernel; 0 = a quarter of the SMs; -1: by H
    int fwd_sync;                   // 1: workers of the forward kernel meet (softly) at every round start
    int chunk_sync;                 // bit 0: same for the recompute GEMM, bit 1: dHidden GEMM, bit 2: dW GEMM
    int logit_stash;                // 1: the loss call keeps the logits of one row block instead of recomputing them
    int l2_hints[UNITY_PROF_CLASSES]; // per GEMM class: GemmArgs::l2_hints
    int wide_acc;                   // 1: dHidden / dW chunk GEMMs may use tiles two MMA blocks wide (CTA pairs only)
    int host_counts;                // 0 (default): stages 2 and 3 never synchronise; 1: they read the K row counts back (one
                                    // stream synchronisation) and skip the launches that would be empty
    int chunk_sync_period[3];       // recompute / dHidden / dW GEMM: rendezvous at every n-th tile of a worker
    long long wait_budget;          // SM clocks after which an in-kernel wait gives up
    int test_drop;                  // test hook: 1 + GEMM class whose producer leaves out one K slab; 0 = off
    int grad_rounds;                // > 0: the recompute GEMM runs on the forward's schedule (rounds of at most this many
                                    // 128-row tiles x vocabulary splits); 0: one tile per unit in raster groups; -1: by H
    int dw_tail;                    // 1: the dW GEMM's last few vocabulary tiles of a chunk run as a launch of narrow tiles
    int grad_runs;                  // recompute GEMM outside rounds: 0: one output tile per unit; n > 0: units are runs of column
                                    // tiles, planned by the kernel so that about n 128-row tiles are in flight; -1: n from H
    int grad_block;                 // blocks of 18944 rows / vocabulary entries one recompute launch covers per side;
                                    // 0: the whole chunk when the launch runs in rounds, else 1
};

namespace {

constexpr size_t kAlign = 256;
// Gradient chunk: 74 row tiles x 74 vocabulary tiles of 256.  With 74 CTA pairs (148 SMs) every chunk GEMM then runs
// a whole number of waves: recompute 74 x 74 tiles, dHidden 74 x ceil(H/256), dW 74 x ceil(H/256).
constexpr int kChunkRows = 74 * kTileM;      // 18944 token rows
constexpr int kChunkVocab = 74 * kTileN;     // 18944 vocabulary entries
// A gradient chunk spans kDefaultChunkMult x kDefaultChunkMult such blocks by default: the dHidden / dW GEMMs then
// contract over twice as many vocabulary entries / rows per output tile and read-modify-write their outputs half as often.
constexpr int kDefaultChunkMult = 2;
constexpr int kSyncCounters = 16384;       // rendezvous counters per call (4 bytes each)
constexpr int kMinChunkRows = 1024;
constexpr int kMinChunkVocab = 1024;

inline size_t up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int fail(unity_ctx* ctx, int code, const char* fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
        va_end(ap);
    }
    return code;
}
#define CUDA_TRY(ctx, expr)                                                                              \
    do {                                                                                                 \
        cudaError_t e_ = (expr);                                                                         \
        if (e_ != cudaSuccess) return fail(ctx, UNITY_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e_)); \
    } while (0)

// Records an event pair around the launches issued during its lifetime when profiling is on.
struct ProfScope {
    unity_ctx* c;
    bool on;
    ProfScope(unity_ctx* ctx, int cls) : c(ctx), on(ctx->profiling != 0) {
        if (!on) return;
        while (c->ev_pool->size() < c->ev_used + 2) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) { on = false; return; }
            c->ev_pool->push_back(e);
        }
        c->ev_class->push_back(cls);
        cudaEventRecord((*c->ev_pool)[c->ev_used], c->stream);
    }
    ~ProfScope() {
        if (!on) return;
        cudaEventRecord((*c->ev_pool)[c->ev_used + 1], c->stream);
        c->ev_used += 2;
    }
};

// Arrival counters of the round rendezvous: one per launch, all cleared at the start of a call.
struct SyncCounters {
    unsigned* base;
    int used, cap;
    unsigned* next() { return used < cap ? base + used++ : nullptr; }   // beyond the array: that launch runs without
};

// Fields every GEMM launch of class `cls` takes from the context: status word, L2 hints, wait bound, test hook and,
// when `sync` is set, a fresh counter for the round rendezvous.
void gemm_common(unity_ctx* ctx, GemmArgs& g, int cls, SyncCounters* counters, bool sync) {
    g.status = ctx->d_status;
    g.l2_hints = ctx->l2_hints[cls];
    g.wait_budget = ctx->wait_budget;
    g.test_drop_slab = ctx->test_drop == cls + 1;
    g.sync_period = cls == UNITY_PROF_FWD_GEMM ? 1 : ctx->chunk_sync_period[cls - 1];
    if (sync && counters) g.round_counter = counters->next();
}

struct Bump {
    char* base;
    size_t off, cap;
    bool ok;
    template <typename T> T* take(size_t n) {
        off = up(off, kAlign);
        T* p = reinterpret_cast<T*>(base + off);
        off += n * sizeof(T);
        if (off > cap) ok = false;
        return p;
    }
};

struct Layout {
    // routing + forward
    int* tok_slot; int* slot_tok; int8_t* tok_model; int* blk_cnt; DevPlan* plan; unsigned* sync_counters;
    __nv_bfloat16* hp; int* target_p; float4* stats; float *row_lse, *row_ent, *row_logp;
    // loss + backward
    float *coef_a, *coef_b, *inv_sums;
    __nv_bfloat16* G; float* dHc;
    long long max_slots, stats_cap;
    int n_blocks, chunk_rows, chunk_vocab;
    size_t bytes;
};

long long max_slots_of(long long n_tok, int K) { return static_cast<long long>(up(n_tok, kTileM)) + static_cast<long long>(kTileM) * K; }

// Carve the workspace.  chunk_rows / chunk_vocab are the wanted gradient chunk sizes (0 = forward only).
// z_chunks > 0: the G scratch holds that many vocabulary chunks side by side (the logit stash of one row block).
Layout carve(char* base, size_t cap, long long n_tok, int H, int V, int K, int n_inv, int chunk_rows, int chunk_vocab,
             bool* fits, int z_chunks = 0) {
    Layout L;
    memset(&L, 0, sizeof(L));
    Bump b{base, 0, cap, true};
    L.max_slots = max_slots_of(n_tok, K);
    L.n_blocks = static_cast<int>((n_tok + kRouteBlock - 1) / kRouteBlock);
    L.stats_cap = 4 * L.max_slots + 94720LL * K;
    L.tok_slot = b.take<int>(n_tok);
    L.slot_tok = b.take<int>(L.max_slots);
    L.tok_model = b.take<int8_t>(n_tok);
    L.blk_cnt = b.take<int>(static_cast<size_t>(L.n_blocks) * K + 1);
    L.plan = b.take<DevPlan>(1);
    L.sync_counters = b.take<unsigned>(kSyncCounters);
    L.hp = b.take<__nv_bfloat16>(static_cast<size_t>(L.max_slots) * H);
    L.target_p = b.take<int>(L.max_slots);
    L.stats = b.take<float4>(L.stats_cap);
    L.row_lse = b.take<float>(L.max_slots);
    L.row_ent = b.take<float>(L.max_slots);
    L.row_logp = b.take<float>(L.max_slots);
    L.chunk_rows = chunk_rows;
    L.chunk_vocab = chunk_vocab;
    if (chunk_rows > 0) {
        L.coef_a = b.take<float>(L.max_slots);
        L.coef_b = b.take<float>(L.max_slots);
        L.inv_sums = b.take<float>(static_cast<size_t>(n_inv) * 9 + 1);
        L.G = b.take<__nv_bfloat16>(static_cast<size_t>(chunk_rows) * chunk_vocab * (z_chunks > 0 ? z_chunks : 1));
        L.dHc = b.take<float>(static_cast<size_t>(chunk_rows) * H);
    }
    L.bytes = up(b.off, kAlign);
    if (fits) *fits = b.ok;
    return L;
}

int wanted_chunk_rows(long long n_tok, int K, int mult = 1) {
    const long long ms = max_slots_of(n_tok, K), want = static_cast<long long>(kChunkRows) * mult;
    return static_cast<int>(ms < want ? ms : want);
}
// Columns of the G scratch: a full chunk plus head-room of kTailTiles tiles, so that a short remainder of the
// vocabulary (V = 152064 is 8 chunks of 18944 plus 512) is absorbed by the last chunk instead of running as a
// chunk of its own, whose GEMMs would be all epilogue.
constexpr int kTailTiles = 8;
int wanted_chunk_vocab(int V, int mult = 1) {
    const long long vp = static_cast<long long>(up(V, kTileN));
    const long long want = static_cast<long long>(kChunkVocab) * mult + kTailTiles * kTileN;
    return static_cast<int>(vp < want ? vp : want);
}

// Regular width of a vocabulary chunk and the number of chunks: all chunks but the last are `base` wide, the last one
// also takes a remainder of up to kTailTiles tiles (its width stays <= cv).
void vocab_chunks(int V, int cv, int* base_out, int* n_out) {
    const int tail = kTailTiles * kTileN;
    const int base = (V > cv && cv > tail + kTileN) ? cv - tail : cv;
    int n = 0;
    for (int v0 = 0, vc = 0; v0 < V; v0 += vc, ++n) {
        vc = V - v0 < base ? V - v0 : base;
        if (V - (v0 + vc) <= tail && base < cv) vc = V - v0;
    }
    *base_out = base;
    *n_out = n;
}
// Row block of the logit stash: 72 row tiles, so that the forward kernel's rounds (24 row tiles x 3 vocabulary splits
// on 74 CTA pairs) are whole.
constexpr int kStashRows = 72 * kTileM;

// Tensor map over a row-major bf16 matrix [rows, inner]; boxes are 64 elements (128 B, one swizzle row) wide and
// box_rows high.  K-major operands use box_rows = kBoxRows (128); MN-major operands use 64 (= kTileK).
int make_tmap(unity_ctx* ctx, CUtensorMap* tm, const void* ptr, uint64_t inner, uint64_t rows, uint64_t pitch_bytes,
              uint32_t box_rows) {
    cuuint64_t dims[2] = {inner, rows};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {64u, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = ctx->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, static_cast<CUtensorMapL2promotion>(ctx->l2_promotion),
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(ctx, UNITY_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d): inner=%llu rows=%llu pitch=%llu", (int)r,
                    (unsigned long long)inner, (unsigned long long)rows, (unsigned long long)pitch_bytes);
    return UNITY_OK;
}

int validate_rows(unity_ctx* ctx, const unity_rows* r) {
    if (!ctx) return UNITY_ERR_INVALID_ARG;
    if (!r) return fail(ctx, UNITY_ERR_INVALID_ARG, "rows is NULL");
    if (r->n_tok < 0 || r->n_inv < 0) return fail(ctx, UNITY_ERR_INVALID_ARG, "negative size");
    if (r->n_tok > 0x7fffff00LL) return fail(ctx, UNITY_ERR_SHAPE, "n_tok too large");
    if (r->K < 1 || r->K > UNITY_MAX_MODELS) return fail(ctx, UNITY_ERR_SHAPE, "K=%d outside [1,%d]", r->K, UNITY_MAX_MODELS);
    if (r->n_roles < 1 || r->n_roles > UNITY_MAX_ROLES)
        return fail(ctx, UNITY_ERR_SHAPE, "n_roles=%d outside [1,%d]", r->n_roles, UNITY_MAX_ROLES);
    if (r->H < 64 || r->H % 64 != 0) return fail(ctx, UNITY_ERR_SHAPE, "H=%d must be a positive multiple of 64", r->H);
    if (r->V < 8 || r->V % 8 != 0) return fail(ctx, UNITY_ERR_SHAPE, "V=%d must be a positive multiple of 8", r->V);
    if (!(r->inv_temperature > 0.f)) return fail(ctx, UNITY_ERR_INVALID_ARG, "inv_temperature must be > 0");
    if (!r->W || !r->role_model) return fail(ctx, UNITY_ERR_INVALID_ARG, "W / role_model is NULL");
    if (r->n_tok > 0 && (!r->hidden || !r->cu_seqlens || !r->inv_role || !r->target || r->n_inv < 1))
        return fail(ctx, UNITY_ERR_INVALID_ARG, "hidden / cu_seqlens / inv_role / target is NULL or n_inv < 1");
    if (reinterpret_cast<uintptr_t>(r->hidden) & 15) return fail(ctx, UNITY_ERR_ALIGNMENT, "hidden not 16-byte aligned");
    for (int k = 0; k < r->K; ++k) {
        if (!r->W[k]) return fail(ctx, UNITY_ERR_INVALID_ARG, "W[%d] is NULL", k);
        if (reinterpret_cast<uintptr_t>(r->W[k]) & 15) return fail(ctx, UNITY_ERR_ALIGNMENT, "W[%d] not 16-byte aligned", k);
    }
    for (int v = 0; v < r->n_roles; ++v)
        if (r->role_model[v] < 0 || r->role_model[v] >= r->K)
            return fail(ctx, UNITY_ERR_INVALID_ARG, "role_model[%d]=%d outside [0,%d)", v, r->role_model[v], r->K);
    return UNITY_OK;
}

// Everything the launches of one call share: the carved workspace, the rendezvous counters, and, only when the host was
// asked to read the row counts back, the padded rows of each model (otherwise -1: not known here).
struct RowPlan {
    Layout L;
    SyncCounters counters;
    FwdPlanParams fwd;
    int rows_known[UNITY_MAX_MODELS];
    long long rows_bound;                 // padded rows a model can have at most: every row of the batch
};

// A round of the forward schedule keeps its hidden rows in L2 while the W tiles stream past.  Where half the machine's
// worth of 256-row tiles (37 on 148 SMs) fits a 45 MB budget (H <= 2368) the rounds are that large: every worker of a
// two-split round then shares its W stream with 36 others.  Measured at H = 896 / 1536: forward +2 %, recompute GEMM
// +19 % / +11 % over rounds of 24 / one tile per unit; at H = 3584 / 5120 such rounds overflow L2 (SM clock -3 %).
bool large_rounds_fit(const unity_ctx* ctx, int H) {
    const long long tiles = ctx->sm_count / 4;
    return tiles * kTileM * H * 2 <= 45ll << 20;
}

// Inputs of the forward planner that the host knows.
FwdPlanParams fwd_params(const unity_ctx* ctx, int V, int H) {
    const int ctas = ctx->ctas[UNITY_PROF_FWD_GEMM];
    FwdPlanParams p;
    p.n_pairs = ctx->sm_count / ctas;
    p.tile_rows = gemm_tile_rows(ctas);
    p.n_tiles = (V + kTileN - 1) / kTileN;
    const int group = ctx->fwd_group >= 0 ? ctx->fwd_group : (large_rounds_fit(ctx, H) ? ctx->sm_count / 2 : 48);
    int gmax = group > 0 ? group / ctas : p.n_pairs / 4;
    if (gmax < 1) gmax = 1;
    if (gmax > p.n_pairs) gmax = p.n_pairs;
    p.gmax = gmax;
    return p;
}

// Optional stash of the scaled logits written by the forward kernel (see GemmArgs::Z).
struct ZStash {
    __nv_bfloat16* Z;
    long long ldz, chunk_stride;
    int chunk_cols, chunks;
};

// LM-head GEMM + online softmax statistics for the rows of `span` (a whole model, or one block of its rows).  The
// kernel derives rows, rounds and splits from the device plan; statistics go to stats (+ the model's base with
// `stats_from_plan`) as [split][row - first row of the span].
int launch_forward(unity_ctx* ctx, const unity_rows* r, RowPlan& P, const RowSpan& span, bool stats_from_plan,
                   const CUtensorMap& tmA, const CUtensorMap& tmB, const ZStash* z) {
    const int ctas = ctx->ctas[UNITY_PROF_FWD_GEMM];
    GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.span = span; g.span_mode = kSpanForward; g.stats_from_plan = stats_from_plan ? 1 : 0; g.fwd = P.fwd;
    g.m_tiles = 1;                                   // set by the kernel
    g.n_tiles = (r->V + kTileN - 1) / kTileN; g.k_iters = r->H / kTileK;
    g.b_row0 = 0; g.a_k0 = 0; g.b_k0 = 0;
    g.n_cols = r->V;
    g.stats = P.L.stats;
    g.target_p = P.L.target_p; g.vocab0 = 0; g.scale = r->inv_temperature;
    if (z) {
        g.Z = z->Z; g.ldz = z->ldz; g.z_chunk_stride = z->chunk_stride; g.z_chunk_cols = z->chunk_cols; g.z_chunks = z->chunks;
        g.g_wide_store = (reinterpret_cast<uintptr_t>(z->Z) % 32 == 0) && (z->ldz * 2 % 32 == 0) && (z->chunk_stride * 2 % 32 == 0) &&
                         (z->chunk_cols * 2 % 32 == 0);
    }
    gemm_common(ctx, g, UNITY_PROF_FWD_GEMM, &P.counters, ctx->fwd_sync != 0);
    // when the host knows the rows it launches exactly the workers a round needs (which CTAs exist decides where they
    // run, and the forward's W streams are sensitive to that: 72 instead of 74 CTA pairs is 10 % faster at H = 3584)
    int workers = 0;
    if (P.rows_known[span.model] >= 0) {
        long long rows = P.rows_known[span.model] - span.row_begin;
        rows = rows < 0 ? 0 : (rows < span.row_cap ? rows : span.row_cap);
        const FwdShape fs = forward_shape(P.fwd, static_cast<int>(rows));
        const int m_tiles = static_cast<int>(rows / P.fwd.tile_rows);
        const int full = (m_tiles < fs.gm ? m_tiles : fs.gm) * fs.splits, last = (m_tiles - fs.last_m0) * fs.last_splits;
        workers = full > last ? full : last;
    }
    ProfScope ps(ctx, UNITY_PROF_FWD_GEMM);
    CUDA_TRY(ctx, launch_gemm(kEpiSoftmaxStats, false, ctas, tmA, tmB, g, ctx->sm_count, ctx->stream, false, workers));
    return UNITY_OK;
}

// Padded rows of model k as far as the host knows: the exact number when it read the counts back, else the bound.
long long rows_of(const RowPlan& P, int k) { return P.rows_known[k] >= 0 ? P.rows_known[k] : P.rows_bound; }

// Routing, packing and the forward sweep: fills per-split softmax statistics for every packed row.
int forward_sweep(unity_ctx* ctx, const unity_rows* r, RowPlan& P, bool run_gemm = true) {
    const Layout& L = P.L;
    cudaStream_t st = ctx->stream;
    int nl = 0;
    P.fwd = fwd_params(ctx, r->V, r->H);
    P.counters = SyncCounters{L.sync_counters, 0, kSyncCounters};
    P.rows_bound = static_cast<long long>(up(r->n_tok, kTileM));
    for (int k = 0; k < UNITY_MAX_MODELS; ++k) P.rows_known[k] = -1;
    CUDA_TRY(ctx, cudaMemsetAsync(L.slot_tok, 0xff, sizeof(int) * L.max_slots, st));
    CUDA_TRY(ctx, cudaMemsetAsync(L.sync_counters, 0, sizeof(unsigned) * kSyncCounters, st));
    RouteArgs ra;
    memset(&ra, 0, sizeof(ra));
    ra.n_tok = r->n_tok; ra.n_inv = r->n_inv; ra.n_roles = r->n_roles; ra.K = r->K; ra.V = r->V;
    ra.cu_seqlens = r->cu_seqlens; ra.inv_role = r->inv_role; ra.target = r->target; ra.tok_mask = r->tok_mask;
    for (int v = 0; v < r->n_roles; ++v) ra.role_model[v] = r->role_model[v];
    ra.n_blocks = L.n_blocks; ra.blk_cnt = L.blk_cnt; ra.plan = L.plan; ra.fwd = P.fwd;
    ra.tok_slot = L.tok_slot; ra.slot_tok = L.slot_tok; ra.tok_model = L.tok_model; ra.status = ctx->d_status;
    CUDA_TRY(ctx, launch_route(ra, st, &nl));
    if (ctx->host_counts) {
        // optional: the host learns the K row counts (a few bytes, one synchronisation) and skips empty launches
        CUDA_TRY(ctx, cudaMemcpyAsync(ctx->h_pinned, L.plan, sizeof(int) * UNITY_MAX_MODELS, cudaMemcpyDeviceToHost, st));
        CUDA_TRY(ctx, cudaStreamSynchronize(st));
        for (int k = 0; k < r->K; ++k) P.rows_known[k] = static_cast<int>(up(ctx->h_pinned[k], kTileM));
    }
    CUDA_TRY(ctx, launch_gather_rows(static_cast<const __nv_bfloat16*>(r->hidden), r->target, L.slot_tok, L.plan, r->K,
                                     L.max_slots, r->H, L.hp, L.target_p, st));
    nl += 1;

    CUtensorMap tmA;
    int rc = make_tmap(ctx, &tmA, L.hp, r->H, L.max_slots, static_cast<uint64_t>(r->H) * 2, kBoxRows);
    if (rc) return rc;
    for (int k = 0; k < r->K && run_gemm; ++k) {
        if (rows_of(P, k) == 0) continue;
        CUtensorMap tmB;
        rc = make_tmap(ctx, &tmB, r->W[k], r->H, r->V, static_cast<uint64_t>(r->H) * 2, kTileN / ctx->ctas[UNITY_PROF_FWD_GEMM]);
        if (rc) return rc;
        const RowSpan whole{L.plan, k, 0, 0x7fffff00};
        rc = launch_forward(ctx, r, P, whole, true, tmA, tmB, nullptr);
        if (rc) return rc;
        nl += 1;
    }
    ctx->launches += nl;
    return UNITY_OK;
}

void fill_token_args(TokenArgs& t, const unity_rows* r, const RowPlan& P) {
    memset(&t, 0, sizeof(t));
    const Layout& L = P.L;
    t.block = RowSpan{L.plan, -1, 0, 0};
    t.plan = L.plan; t.fwd = P.fwd; t.max_slots = L.max_slots;
    t.K = r->K; t.n_roles = r->n_roles; t.n_inv = r->n_inv; t.n_tok = r->n_tok;
    t.stats = L.stats;
    t.slot_tok = L.slot_tok; t.tok_slot = L.tok_slot; t.tok_model = L.tok_model;
    t.scale = r->inv_temperature;
    t.row_lse = L.row_lse; t.row_ent = L.row_ent; t.row_logp = L.row_logp;
    t.cu_seqlens = r->cu_seqlens; t.inv_role = r->inv_role;
    for (int v = 0; v < r->n_roles; ++v) t.role_model[v] = r->role_model[v];
}

}  // namespace

// ================================================================================================
extern "C" {

int unity_create(unity_ctx** out, int device, void* cuda_stream, void* workspace, size_t workspace_bytes) {
    if (!out) return UNITY_ERR_INVALID_ARG;
    *out = nullptr;
    if (workspace_bytes > 0 && !workspace) return UNITY_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return UNITY_ERR_ALIGNMENT;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { cudaGetLastError(); return UNITY_ERR_CUDA; }
    if (prop.major != 10) return UNITY_ERR_UNSUPPORTED_ARCH;
    if (cudaSetDevice(device) != cudaSuccess) return UNITY_ERR_CUDA;
    unity_ctx* c = new (std::nothrow) unity_ctx();
    if (!c) return UNITY_ERR_CUDA;
    memset(c, 0, sizeof(*c));
    c->device = device;
    c->stream = static_cast<cudaStream_t>(cuda_stream);
    c->ws = static_cast<char*>(workspace);
    c->ws_bytes = workspace_bytes;
    c->sm_count = prop.multiProcessorCount;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess) {
        delete c;
        return UNITY_ERR_CUDA;
    }
    c->encode = reinterpret_cast<EncodeTiledFn>(fn);
    c->ctas[UNITY_PROF_FWD_GEMM] = 2;
    c->ctas[UNITY_PROF_GRAD_GEMM] = 2;
    c->ctas[UNITY_PROF_DH_GEMM] = 2;
    c->ctas[UNITY_PROF_DW_GEMM] = 2;
    c->l2_promotion = 3;
    c->chunk_group[0] = 40;          // recompute: least DRAM traffic of 32 / 40 / 48 / 64 (3.9 bytes per logit), same time
    c->chunk_group[1] = c->chunk_group[2] = 32;
    c->fwd_group = -1;
    c->fwd_sync = 1;
    c->chunk_sync = 7;
    c->chunk_rows_mult = kDefaultChunkMult;
    c->chunk_vocab_mult = kDefaultChunkMult;
    c->wide_acc = 1;
    // forward / recompute: the round's hidden rows are kept (evict last) while the W stream passes (evict first); the
    // logit-gradient chunk is written evict-first, it is far larger than L2 and not read again by the same kernel
    c->l2_hints[UNITY_PROF_FWD_GEMM] = 2 | (1 << 2);
    c->l2_hints[UNITY_PROF_GRAD_GEMM] = 2 | (1 << 2) | (1 << 4);
    c->l2_hints[UNITY_PROF_DH_GEMM] = 0;
    c->l2_hints[UNITY_PROF_DW_GEMM] = 0;
    c->logit_stash = 0;
    c->chunk_sync_period[0] = c->chunk_sync_period[1] = c->chunk_sync_period[2] = 1;
    c->host_counts = 0;
    c->wait_budget = kWaitBudgetCycles;
    c->test_drop = 0;
    c->grad_rounds = -1;
    c->grad_runs = -1;
    c->dw_tail = 1;
    c->grad_block = 0;
    c->ev_pool = new (std::nothrow) std::vector<cudaEvent_t>();
    c->ev_class = new (std::nothrow) std::vector<int>();
    if (cudaMalloc(&c->d_status, 256) != cudaSuccess || cudaMallocHost(&c->h_pinned, 4096) != cudaSuccess ||
        cudaMemset(c->d_status, 0, 256) != cudaSuccess || gemm_set_attributes() != cudaSuccess) {
        if (c->d_status) cudaFree(c->d_status);
        if (c->h_pinned) cudaFreeHost(c->h_pinned);
        delete c;
        cudaGetLastError();
        return UNITY_ERR_CUDA;
    }
    *out = c;
    return UNITY_OK;
}

int unity_destroy(unity_ctx* ctx) {
    if (!ctx) return UNITY_ERR_INVALID_ARG;
    cudaSetDevice(ctx->device);
    cudaStreamSynchronize(ctx->stream);
    cudaFree(ctx->d_status);
    cudaFreeHost(ctx->h_pinned);
    if (ctx->ev_pool) for (cudaEvent_t e : *ctx->ev_pool) cudaEventDestroy(e);
    delete ctx->ev_pool;
    delete ctx->ev_class;
    delete ctx;
    return UNITY_OK;
}

size_t unity_workspace_bytes(int64_t n_tok, int32_t H, int32_t V, int32_t K, int32_t n_inv) {
    if (n_tok < 0 || H <= 0 || V <= 0 || K <= 0 || n_inv < 0) return 0;
    return carve(nullptr, ~size_t(0), n_tok, H, V, K, n_inv, wanted_chunk_rows(n_tok, K, kDefaultChunkMult),
                 wanted_chunk_vocab(V, kDefaultChunkMult), nullptr).bytes;
}

size_t unity_advantage_workspace_bytes(int32_t n_inv, int32_t n_groups, int32_t n_roles) {
    if (n_inv < 0 || n_groups < 1 || n_roles < 1) return 0;
    Bump b{nullptr, 0, ~size_t(0), true};
    b.take<float>(static_cast<size_t>(n_inv) + 4);
    b.take<int>(static_cast<size_t>(n_inv) + 4);
    b.take<char>(advantage_table_bytes(static_cast<long long>(n_groups) * n_roles));
    return up(b.off, kAlign);
}

size_t unity_workspace_hint(int64_t n_tok, int32_t H, int32_t V, int32_t K) {
    if (n_tok < 0 || n_tok > 0x7fffff00LL) return 0;
    return unity_workspace_bytes(n_tok, H, V, K, static_cast<int32_t>(n_tok));
}

size_t unity_workspace_bytes_stash(int64_t n_tok, int32_t H, int32_t V, int32_t K, int32_t n_inv) {
    if (n_tok < 0 || H <= 0 || V <= 0 || K <= 0 || n_inv < 0) return 0;
    int cr = wanted_chunk_rows(n_tok, K);
    if (cr > kStashRows) cr = kStashRows;
    const int cv = wanted_chunk_vocab(V, kDefaultChunkMult);
    int base, n;
    vocab_chunks(V, cv, &base, &n);
    const size_t a = carve(nullptr, ~size_t(0), n_tok, H, V, K, n_inv, cr, cv, nullptr, n).bytes;
    const size_t b = unity_workspace_bytes(n_tok, H, V, K, n_inv);
    return a > b ? a : b;
}

size_t unity_workspace_min_bytes(int64_t n_tok, int32_t H, int32_t V, int32_t K, int32_t n_inv) {
    if (n_tok < 0 || H <= 0 || V <= 0 || K <= 0 || n_inv < 0) return 0;
    int cr = wanted_chunk_rows(n_tok, K), cv = wanted_chunk_vocab(V);
    if (cr > kMinChunkRows) cr = kMinChunkRows;
    if (cv > kMinChunkVocab) cv = kMinChunkVocab;
    return carve(nullptr, ~size_t(0), n_tok, H, V, K, n_inv, cr, cv, nullptr).bytes;
}

int unity_check_status(unity_ctx* ctx) {
    if (!ctx) return UNITY_ERR_INVALID_ARG;
    CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    CUDA_TRY(ctx, cudaMemcpyAsync(ctx->h_pinned + 512, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
    CUDA_TRY(ctx, cudaMemsetAsync(ctx->d_status, 0, sizeof(int), ctx->stream));
    CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream));
    const int bits = ctx->h_pinned[512];
    if (bits & kStatusTimeout) return fail(ctx, UNITY_ERR_TIMEOUT, "a bounded in-kernel wait expired");
    if (bits & kStatusBadIndex) return fail(ctx, UNITY_ERR_BAD_INDEX, "an index in the data was out of range (row / invocation masked)");
    return UNITY_OK;
}

const char* unity_last_error(const unity_ctx* ctx) { return ctx ? ctx->err : "null context"; }

int64_t unity_launch_count(const unity_ctx* ctx) { return ctx ? ctx->launches : 0; }

int unity_set_option(unity_ctx* ctx, int option, int value) {
    if (!ctx) return UNITY_ERR_INVALID_ARG;
    if (option >= UNITY_OPT_CTAS_FWD && option <= UNITY_OPT_CTAS_DW) {
        if (value != 1 && value != 2) return fail(ctx, UNITY_ERR_INVALID_ARG, "CTAs per tile must be 1 or 2");
        ctx->ctas[option - UNITY_OPT_CTAS_FWD] = value;
        return UNITY_OK;
    }
    if (option == UNITY_OPT_L2_PROMOTION && value >= 0 && value <= 3) { ctx->l2_promotion = value; return UNITY_OK; }
    if (option == UNITY_OPT_CHUNK_GROUP && value >= 2 && value <= 148) {
        ctx->chunk_group[0] = ctx->chunk_group[1] = ctx->chunk_group[2] = value;
        return UNITY_OK;
    }
    if (option >= UNITY_OPT_GROUP_GRAD && option <= UNITY_OPT_GROUP_DW && value >= 2 && value <= 148) {
        ctx->chunk_group[option - UNITY_OPT_GROUP_GRAD] = value;
        return UNITY_OK;
    }
    if (option == UNITY_OPT_FWD_SYNC && (value == 0 || value == 1)) { ctx->fwd_sync = value; return UNITY_OK; }
    if (option == UNITY_OPT_CHUNK_SYNC && value >= 0 && value <= 7) { ctx->chunk_sync = value; return UNITY_OK; }
    if (option == UNITY_OPT_FWD_GROUP && value >= -1 && value <= 148) { ctx->fwd_group = value; return UNITY_OK; }
    if (option == UNITY_OPT_CHUNK_ROWS && value >= 1 && value <= 8) { ctx->chunk_rows_mult = value; return UNITY_OK; }
    if (option == UNITY_OPT_CHUNK_VOCAB && value >= 1 && value <= 8) { ctx->chunk_vocab_mult = value; return UNITY_OK; }
    if (option == UNITY_OPT_LOGIT_STASH && (value == 0 || value == 1)) { ctx->logit_stash = value; return UNITY_OK; }
    if (option >= UNITY_OPT_L2_HINTS_FWD && option < UNITY_OPT_L2_HINTS_FWD + UNITY_PROF_CLASSES && value >= 0 && value < 64) {
        ctx->l2_hints[option - UNITY_OPT_L2_HINTS_FWD] = value;
        return UNITY_OK;
    }
    if (option == UNITY_OPT_WIDE_ACC && (value == 0 || value == 1)) { ctx->wide_acc = value; return UNITY_OK; }
    if (option >= UNITY_OPT_SYNC_PERIOD_GRAD && option <= UNITY_OPT_SYNC_PERIOD_DW && value >= 1 && value <= 1024) {
        ctx->chunk_sync_period[option - UNITY_OPT_SYNC_PERIOD_GRAD] = value;
        return UNITY_OK;
    }
    if (option == UNITY_OPT_HOST_COUNTS && (value == 0 || value == 1)) { ctx->host_counts = value; return UNITY_OK; }
    if (option == UNITY_OPT_GRAD_ROUNDS && value >= -1 && value <= 148) { ctx->grad_rounds = value; return UNITY_OK; }
    if (option == UNITY_OPT_GRAD_RUNS && value >= -1 && value <= 148) { ctx->grad_runs = value; return UNITY_OK; }
    if (option == UNITY_OPT_DW_TAIL && (value == 0 || value == 1)) { ctx->dw_tail = value; return UNITY_OK; }
    if (option == UNITY_OPT_GRAD_BLOCK && value >= 0 && value <= 8) { ctx->grad_block = value; return UNITY_OK; }
    if (option == UNITY_OPT_WAIT_KCYCLES && value >= 1) {
        ctx->wait_budget = static_cast<long long>(value) * 1000;
        if (ctx->wait_budget > 1000000) ctx->test_drop = 0;      // the test hook lives only under a short bound
        return UNITY_OK;
    }
    if (option == UNITY_OPT_TEST_DROP_SLAB && value >= 0 && value <= UNITY_PROF_CLASSES) {
        if (value != 0 && ctx->wait_budget > 1000000)
            return fail(ctx, UNITY_ERR_INVALID_ARG, "UNITY_OPT_TEST_DROP_SLAB needs UNITY_OPT_WAIT_KCYCLES <= 1000 first");
        ctx->test_drop = value;
        return UNITY_OK;
    }
    return fail(ctx, UNITY_ERR_INVALID_ARG, "unknown option %d or value %d out of range", option, value);
}

int unity_set_profiling(unity_ctx* ctx, int enable) {
    if (!ctx || !ctx->ev_pool || !ctx->ev_class) return UNITY_ERR_INVALID_ARG;
    ctx->profiling = enable != 0;
    ctx->ev_used = 0;
    ctx->ev_class->clear();
    return UNITY_OK;
}

int unity_get_profile(unity_ctx* ctx, double* ms, int64_t* launches) {
    if (!ctx || !ms || !launches || !ctx->ev_pool) return UNITY_ERR_INVALID_ARG;
    for (int i = 0; i < UNITY_PROF_CLASSES; ++i) { ms[i] = 0.0; launches[i] = 0; }
    CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    CUDA_TRY(ctx, cudaStreamSynchronize(ctx->stream));
    for (size_t i = 0; i < ctx->ev_class->size(); ++i) {
        float t = 0.f;
        CUDA_TRY(ctx, cudaEventElapsedTime(&t, (*ctx->ev_pool)[2 * i], (*ctx->ev_pool)[2 * i + 1]));
        const int cls = (*ctx->ev_class)[i];
        ms[cls] += t;
        launches[cls] += 1;
    }
    ctx->ev_used = 0;
    ctx->ev_class->clear();
    return UNITY_OK;
}

// ------------------------------------------------------------------------------------------------
int unity_role_advantage(unity_ctx* ctx, int32_t n_inv, int32_t n_traj, int32_t n_roles, int32_t n_groups,
                         const int32_t* inv_role, const int32_t* inv_group, const int32_t* inv_traj,
                         const float* r_node, const float* r_turn, const float* r_traj, const float* lam,
                         const unity_adv_params* params, int64_t n_tok, const int64_t* cu_seqlens,
                         const uint8_t* tok_mask, float* adv_inv, float* adv_tok, float* seg_mean, float* seg_std) {
    if (!ctx) return UNITY_ERR_INVALID_ARG;
    if (n_inv < 0 || n_traj < 0 || n_tok < 0) return fail(ctx, UNITY_ERR_INVALID_ARG, "negative size");
    if (n_roles < 1 || n_roles > UNITY_MAX_ROLES) return fail(ctx, UNITY_ERR_SHAPE, "n_roles=%d outside [1,%d]", n_roles, UNITY_MAX_ROLES);
    if (n_groups < 1 || static_cast<long long>(n_groups) * n_roles > (1 << 24))
        return fail(ctx, UNITY_ERR_SHAPE, "n_groups*n_roles outside [1, 2^24]");
    if (n_inv > 0 && (!inv_role || !inv_group || !adv_inv)) return fail(ctx, UNITY_ERR_INVALID_ARG, "inv_role / inv_group / adv_inv is NULL");
    if (r_traj && n_inv > 0 && !inv_traj) return fail(ctx, UNITY_ERR_INVALID_ARG, "r_traj given without inv_traj");
    if (n_tok > 0 && (!cu_seqlens || !adv_tok || n_inv < 1)) return fail(ctx, UNITY_ERR_INVALID_ARG, "cu_seqlens / adv_tok is NULL or n_inv < 1");
    const float eps = params ? params->eps : 1e-6f;
    const int ddof = params ? params->ddof : 0;
    if (!(eps >= 0.f) || (ddof != 0 && ddof != 1)) return fail(ctx, UNITY_ERR_INVALID_ARG, "eps must be >= 0 and ddof 0 or 1");
    CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    Bump b{ctx->ws, 0, ctx->ws_bytes, true};
    AdvArgs a;
    memset(&a, 0, sizeof(a));
    a.r_scratch = b.take<float>(n_inv + 4);
    a.seg_scratch = b.take<int>(n_inv + 4);
    a.seg_table = b.take<char>(advantage_table_bytes(static_cast<long long>(n_groups) * n_roles));
    if (!b.ok)
        return fail(ctx, UNITY_ERR_WORKSPACE, "workspace too small: stage 1 needs %zu bytes (unity_advantage_workspace_bytes)", b.off);
    a.n_inv = n_inv; a.n_traj = n_traj; a.n_roles = n_roles; a.n_groups = n_groups;
    a.inv_role = inv_role; a.inv_group = inv_group; a.inv_traj = inv_traj;
    a.r_node = r_node; a.r_turn = r_turn; a.r_traj = r_traj;
    a.has_lam = lam != nullptr;
    if (lam) memcpy(a.lam, lam, sizeof(float) * 3 * n_roles);
    a.eps = eps; a.ddof = ddof; a.n_tok = n_tok; a.cu_seqlens = cu_seqlens; a.tok_mask = tok_mask;
    a.adv_inv = adv_inv; a.adv_tok = adv_tok; a.seg_mean = seg_mean; a.seg_std = seg_std;
    a.status = ctx->d_status;
    int nl = 0;
    CUDA_TRY(ctx, launch_advantage(a, ctx->stream, &nl));
    ctx->launches += nl;
    return UNITY_OK;
}

// ------------------------------------------------------------------------------------------------
int unity_reward_assembly(unity_ctx* ctx, int32_t n_inv, int32_t n_traj, int32_t n_roles, int32_t max_turns,
                          const int32_t* inv_role, const int32_t* inv_traj, const int32_t* inv_turn, const float* score,
                          const int32_t* n_scores, const uint8_t* inv_end, const unity_reward_rule* rules,
                          float* r_turn) {
    if (!ctx) return UNITY_ERR_INVALID_ARG;
    if (n_inv < 0 || n_traj < 0 || max_turns < 1) return fail(ctx, UNITY_ERR_INVALID_ARG, "negative size or max_turns < 1");
    if (n_roles < 1 || n_roles > UNITY_MAX_ROLES) return fail(ctx, UNITY_ERR_SHAPE, "n_roles=%d outside [1,%d]", n_roles, UNITY_MAX_ROLES);
    if (!rules) return fail(ctx, UNITY_ERR_INVALID_ARG, "rules is NULL");
    if (n_inv > 0 && (!inv_role || !inv_traj || !inv_turn || !score || !r_turn))
        return fail(ctx, UNITY_ERR_INVALID_ARG, "inv_role / inv_traj / inv_turn / score / r_turn is NULL");
    RewardArgs a;
    memset(&a, 0, sizeof(a));
    for (int v = 0; v < n_roles; ++v) {
        if (rules[v].mode < UNITY_RULE_NONE || rules[v].mode > UNITY_RULE_MARGINAL)
            return fail(ctx, UNITY_ERR_INVALID_ARG, "rules[%d].mode must be 0, 1 or 2", v);
        a.mode[v] = rules[v].mode;
        a.shift[v] = rules[v].shift;
    }
    if (n_inv == 0) return UNITY_OK;
    CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    a.n_inv = n_inv; a.n_traj = n_traj; a.n_roles = n_roles; a.max_turns = max_turns;
    a.inv_role = inv_role; a.inv_traj = inv_traj; a.inv_turn = inv_turn; a.score = score; a.n_scores = n_scores;
    a.inv_end = inv_end; a.r_turn = r_turn; a.status = ctx->d_status;
    CUDA_TRY(ctx, launch_reward_assembly(a, ctx->stream));
    ctx->launches += 1;
    return UNITY_OK;
}

// ------------------------------------------------------------------------------------------------
int unity_gae(unity_ctx* ctx, int32_t n_inv, int64_t n_tok, const int64_t* cu_seqlens, const float* rewards,
              const float* values, const uint8_t* tok_mask, float gamma, float lam, float* advantages, float* returns) {
    if (!ctx) return UNITY_ERR_INVALID_ARG;
    if (n_inv < 0 || n_tok < 0) return fail(ctx, UNITY_ERR_INVALID_ARG, "negative size");
    if (n_tok > 0 && (n_inv < 1 || !cu_seqlens || !rewards || !values || !advantages || !returns))
        return fail(ctx, UNITY_ERR_INVALID_ARG, "cu_seqlens / rewards / values / advantages / returns is NULL or n_inv < 1");
    if (!(gamma >= 0.f && gamma <= 1.f) || !(lam >= 0.f && lam <= 1.f))
        return fail(ctx, UNITY_ERR_INVALID_ARG, "gamma and lambda must lie in [0, 1]");
    if (n_tok == 0) return UNITY_OK;
    CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    CUDA_TRY(ctx, launch_gae(n_inv, cu_seqlens, rewards, values, tok_mask, gamma, lam, advantages, returns, ctx->stream));
    ctx->launches += 1;
    return UNITY_OK;
}

// ------------------------------------------------------------------------------------------------
int unity_value_loss_fwd_bwd(unity_ctx* ctx, int32_t n_inv, int32_t n_roles, int32_t K, int64_t n_tok,
                             const int64_t* cu_seqlens, const int32_t* inv_role, const int32_t* role_model,
                             const uint8_t* tok_mask, const float* values, const float* old_values,
                             const float* returns, float clip_v, const float* norm, float* loss, float* clip_frac,
                             float* tok_loss, float* dvalues) {
    if (!ctx) return UNITY_ERR_INVALID_ARG;
    if (n_inv < 0 || n_tok < 0) return fail(ctx, UNITY_ERR_INVALID_ARG, "negative size");
    if (n_roles < 1 || n_roles > UNITY_MAX_ROLES) return fail(ctx, UNITY_ERR_SHAPE, "n_roles=%d outside [1,%d]", n_roles, UNITY_MAX_ROLES);
    if (K < 1 || K > UNITY_MAX_MODELS) return fail(ctx, UNITY_ERR_SHAPE, "K=%d outside [1,%d]", K, UNITY_MAX_MODELS);
    if (!role_model || !loss) return fail(ctx, UNITY_ERR_INVALID_ARG, "role_model / loss is NULL");
    if (!(clip_v >= 0.f)) return fail(ctx, UNITY_ERR_INVALID_ARG, "clip_v must be >= 0");
    if (n_inv > 0 && (!cu_seqlens || !inv_role)) return fail(ctx, UNITY_ERR_INVALID_ARG, "cu_seqlens / inv_role is NULL");
    if (n_tok > 0 && (n_inv < 1 || !values || !old_values || !returns || !dvalues))
        return fail(ctx, UNITY_ERR_INVALID_ARG, "values / old_values / returns / dvalues is NULL or n_inv < 1");
    ValueArgs a;
    memset(&a, 0, sizeof(a));
    for (int k = 0; k < K; ++k) {
        if (norm && !(norm[k] > 0.f)) return fail(ctx, UNITY_ERR_INVALID_ARG, "norm[%d] must be > 0", k);
        if (norm) a.norm[k] = norm[k];
    }
    for (int v = 0; v < n_roles; ++v) a.role_model[v] = role_model[v];
    CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    Bump b{ctx->ws, 0, ctx->ws_bytes, true};
    a.model_cnt = reinterpret_cast<unsigned long long*>(b.take<char>(value_counters_bytes()));
    a.tickets = reinterpret_cast<int*>(a.model_cnt + UNITY_MAX_MODELS);
    a.partial = b.take<float>(static_cast<size_t>(UNITY_MAX_MODELS) * kValueSlices * 2);
    a.inv_sums = b.take<float>(static_cast<size_t>(n_inv) * 3 + 4);
    if (!b.ok) return fail(ctx, UNITY_ERR_WORKSPACE, "workspace too small: need %zu bytes", b.off);
    a.n_inv = n_inv; a.n_roles = n_roles; a.K = K;
    a.cu_seqlens = cu_seqlens; a.inv_role = inv_role; a.tok_mask = tok_mask;
    a.values = values; a.old_values = old_values; a.returns = returns;
    a.clip_v = clip_v; a.has_norm = norm != nullptr;
    a.vec_ok = ((reinterpret_cast<uintptr_t>(values) | reinterpret_cast<uintptr_t>(old_values) |
                 reinterpret_cast<uintptr_t>(returns) | reinterpret_cast<uintptr_t>(dvalues) |
                 reinterpret_cast<uintptr_t>(tok_loss)) & 15) == 0 && (reinterpret_cast<uintptr_t>(tok_mask) & 3) == 0;
    a.loss = loss; a.clip_frac = clip_frac; a.tok_loss = tok_loss; a.dvalues = dvalues;
    a.status = ctx->d_status;
    int nl = 0;
    CUDA_TRY(ctx, launch_value_loss(a, ctx->stream, &nl));
    ctx->launches += nl;
    return UNITY_OK;
}

// ------------------------------------------------------------------------------------------------
int unity_ready_batch_plan(unity_ctx* ctx, int32_t n_inv, int32_t n_traj, int32_t n_roles, int32_t K,
                           const int64_t* cu_seqlens, const int32_t* inv_role, const int32_t* inv_traj,
                           const uint8_t* traj_done, const int32_t* role_model, const unity_batch_params* params,
                           int32_t* order, int64_t* out_cu_seqlens, int32_t* model_offsets, int32_t* part_offsets,
                           int64_t* totals) {
    if (!ctx) return UNITY_ERR_INVALID_ARG;
    if (n_inv < 0 || n_traj < 0) return fail(ctx, UNITY_ERR_INVALID_ARG, "negative size");
    if (n_roles < 1 || n_roles > UNITY_MAX_ROLES) return fail(ctx, UNITY_ERR_SHAPE, "n_roles=%d outside [1,%d]", n_roles, UNITY_MAX_ROLES);
    if (K < 1 || K > UNITY_MAX_MODELS) return fail(ctx, UNITY_ERR_SHAPE, "K=%d outside [1,%d]", K, UNITY_MAX_MODELS);
    if (!params || !role_model || !out_cu_seqlens || !model_offsets || !part_offsets || !totals)
        return fail(ctx, UNITY_ERR_INVALID_ARG, "params / role_model / out_cu_seqlens / model_offsets / part_offsets / totals is NULL");
    if (params->n_parts < 1 || params->n_parts > 65536 || params->pad_to < 1)
        return fail(ctx, UNITY_ERR_INVALID_ARG, "n_parts must lie in [1, 65536] and pad_to must be >= 1");
    if (n_inv > 0 && (!cu_seqlens || !inv_role || !inv_traj || !traj_done || !order))
        return fail(ctx, UNITY_ERR_INVALID_ARG, "cu_seqlens / inv_role / inv_traj / traj_done / order is NULL");
    BatchArgs a;
    memset(&a, 0, sizeof(a));
    for (int v = 0; v < n_roles; ++v) {
        if (role_model[v] < -1 || role_model[v] >= K) return fail(ctx, UNITY_ERR_INVALID_ARG, "role_model[%d]=%d outside [-1,%d)", v, role_model[v], K);
        a.role_model[v] = role_model[v];
    }
    CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    a.n_inv = n_inv; a.n_traj = n_traj; a.n_roles = n_roles; a.K = K;
    a.n_parts = params->n_parts; a.pad_to = params->pad_to;
    batch_keys(params->seed, n_inv, &a);
    a.n_blocks = (n_inv + batch_block() - 1) / batch_block();
    Bump b{ctx->ws, 0, ctx->ws_bytes, true};
    a.model_tok = b.take<long long>(UNITY_MAX_MODELS + 1);
    a.pos_inv = b.take<int>(n_inv);
    a.pos_model = b.take<int8_t>(n_inv);
    a.blk_cnt = b.take<int>(static_cast<size_t>(a.n_blocks) * K);
    a.blk_tok = b.take<long long>(static_cast<size_t>(a.n_blocks) * K);
    if (!b.ok) return fail(ctx, UNITY_ERR_WORKSPACE, "workspace too small: need %zu bytes", b.off);
    a.cu_seqlens = cu_seqlens; a.inv_role = inv_role; a.inv_traj = inv_traj; a.traj_done = traj_done;
    a.order = order; a.out_cu = out_cu_seqlens; a.model_offsets = model_offsets; a.part_offsets = part_offsets;
    a.totals = reinterpret_cast<long long*>(totals);
    a.status = ctx->d_status;
    int nl = 0;
    CUDA_TRY(ctx, launch_batch_plan(a, ctx->stream, &nl));
    ctx->launches += nl;
    return UNITY_OK;
}

int unity_ready_batch_gather(unity_ctx* ctx, int32_t n_inv, int64_t n_tok_src, const int32_t* order,
                             const int64_t* src_cu_seqlens, const int64_t* out_cu_seqlens, const int64_t* totals,
                             int64_t row_bytes, const void* src, void* dst, const void* pad_value, int32_t pad_bytes) {
    if (!ctx) return UNITY_ERR_INVALID_ARG;
    if (n_inv < 0 || n_tok_src < 0 || row_bytes < 1) return fail(ctx, UNITY_ERR_INVALID_ARG, "negative size or row_bytes < 1");
    if (pad_bytes != 1 && pad_bytes != 2 && pad_bytes != 4 && pad_bytes != 8)
        return fail(ctx, UNITY_ERR_INVALID_ARG, "pad_bytes must be 1, 2, 4 or 8");
    if (row_bytes % pad_bytes) return fail(ctx, UNITY_ERR_INVALID_ARG, "pad_bytes must divide row_bytes");
    if (n_inv == 0) return UNITY_OK;
    if (!order || !src_cu_seqlens || !out_cu_seqlens || !totals || !dst || (n_tok_src > 0 && !src))
        return fail(ctx, UNITY_ERR_INVALID_ARG, "order / src_cu_seqlens / out_cu_seqlens / totals / src / dst is NULL");
    int unit = 16;
    while (unit > 1 && row_bytes % unit) unit >>= 1;
    if (unit < pad_bytes || (reinterpret_cast<uintptr_t>(src) % unit) || (reinterpret_cast<uintptr_t>(dst) % unit))
        return fail(ctx, UNITY_ERR_ALIGNMENT, "src / dst must be aligned to %d bytes for rows of %lld bytes", unit,
                    static_cast<long long>(row_bytes));
    GatherArgs g;
    memset(&g, 0, sizeof(g));
    g.n_inv = n_inv; g.order = order; g.src_cu = src_cu_seqlens; g.out_cu = out_cu_seqlens;
    g.totals = reinterpret_cast<const long long*>(totals);
    g.row_bytes = row_bytes; g.unit_bytes = unit; g.avg_len = n_tok_src / n_inv + 1;
    g.src = src; g.dst = dst; g.pad_bytes = pad_bytes;
    if (pad_value) memcpy(g.pad, pad_value, pad_bytes);
    CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    CUDA_TRY(ctx, launch_batch_gather(g, ctx->stream));
    ctx->launches += 1;
    return UNITY_OK;
}

int unity_align_rewards(unity_ctx* ctx, int32_t n_inv, int64_t n_tok, const int64_t* cu_seqlens,
                        const uint8_t* tok_mask, const float* r_inv, float* tok_reward) {
    if (!ctx) return UNITY_ERR_INVALID_ARG;
    if (n_inv < 0 || n_tok < 0) return fail(ctx, UNITY_ERR_INVALID_ARG, "negative size");
    if (n_inv > 0 && (!cu_seqlens || !r_inv)) return fail(ctx, UNITY_ERR_INVALID_ARG, "cu_seqlens / r_inv is NULL");
    if (n_tok > 0 && (n_inv < 1 || !tok_reward)) return fail(ctx, UNITY_ERR_INVALID_ARG, "tok_reward is NULL or n_inv < 1");
    if (n_inv == 0) return UNITY_OK;
    CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    CUDA_TRY(ctx, launch_align_rewards(n_inv, cu_seqlens, tok_mask, r_inv, tok_reward, ctx->stream));
    ctx->launches += 1;
    return UNITY_OK;
}

// ------------------------------------------------------------------------------------------------
int unity_logprob_fwd(unity_ctx* ctx, const unity_rows* rows, float* logp, float* entropy, float* lse) {
    int rc = validate_rows(ctx, rows);
    if (rc) return rc;
    if (rows->n_tok > 0 && !logp) return fail(ctx, UNITY_ERR_INVALID_ARG, "logp is NULL");
    if (rows->n_tok == 0) return UNITY_OK;
    CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    RowPlan P;
    bool fits = false;
    P.L = carve(ctx->ws, ctx->ws_bytes, rows->n_tok, rows->H, rows->V, rows->K, rows->n_inv, 0, 0, &fits);
    if (!fits) return fail(ctx, UNITY_ERR_WORKSPACE, "workspace too small: need %zu bytes, have %zu", P.L.bytes, ctx->ws_bytes);
    cudaStream_t st = ctx->stream;
    CUDA_TRY(ctx, cudaMemsetAsync(logp, 0, sizeof(float) * rows->n_tok, st));
    if (entropy) CUDA_TRY(ctx, cudaMemsetAsync(entropy, 0, sizeof(float) * rows->n_tok, st));
    if (lse) CUDA_TRY(ctx, cudaMemsetAsync(lse, 0, sizeof(float) * rows->n_tok, st));
    rc = forward_sweep(ctx, rows, P);
    if (rc) return rc;
    TokenArgs t;
    fill_token_args(t, rows, P);
    t.logp = logp; t.entropy = entropy; t.lse = lse;
    int nl = 0;
    CUDA_TRY(ctx, launch_finish_forward(t, false, st, &nl));
    ctx->launches += nl;
    return UNITY_OK;
}

// ------------------------------------------------------------------------------------------------
int unity_ppo_loss_fwd_bwd(unity_ctx* ctx, const unity_rows* rows, const unity_ppo_params* params,
                           const float* old_logp, const float* ref_logp, const float* adv_tok, float* loss,
                           float* metrics, float* logp, float* entropy, float* tok_loss, void* dHidden,
                           void* const* dW) {
    int rc = validate_rows(ctx, rows);
    if (rc) return rc;
    if (!params || !loss || !dW) return fail(ctx, UNITY_ERR_INVALID_ARG, "params / loss / dW is NULL");
    if (params->kl_mode < 1 || params->kl_mode > 3) return fail(ctx, UNITY_ERR_INVALID_ARG, "kl_mode must be 1, 2 or 3");
    if (!(params->clip_lo >= 0.f) || !(params->clip_hi >= 0.f)) return fail(ctx, UNITY_ERR_INVALID_ARG, "clip ranges must be >= 0");
    if (rows->n_tok > 0 && (!old_logp || !ref_logp || !adv_tok || !dHidden))
        return fail(ctx, UNITY_ERR_INVALID_ARG, "old_logp / ref_logp / adv_tok / dHidden is NULL");
    if (reinterpret_cast<uintptr_t>(dHidden) & 15) return fail(ctx, UNITY_ERR_ALIGNMENT, "dHidden not 16-byte aligned");
    const int K = rows->K, H = rows->H, V = rows->V;
    for (int k = 0; k < K; ++k) {
        if (!dW[k]) return fail(ctx, UNITY_ERR_INVALID_ARG, "dW[%d] is NULL", k);
        if (reinterpret_cast<uintptr_t>(dW[k]) & 15) return fail(ctx, UNITY_ERR_ALIGNMENT, "dW[%d] not 16-byte aligned", k);
        if (params->norm && !(params->norm[k] > 0.f)) return fail(ctx, UNITY_ERR_INVALID_ARG, "norm[%d] must be > 0", k);
    }
    CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    cudaStream_t st = ctx->stream;

    // On-policy shortcut: when the caller hands in logp / entropy / lse of THESE weights on THESE rows (from
    // unity_logprob_fwd), the forward sweep over the vocabulary is skipped; the backward still recomputes the logits.
    const bool have_fwd = params->logp_in && params->entropy_in && params->lse_in;
    if (!have_fwd && (params->logp_in || params->entropy_in || params->lse_in))
        return fail(ctx, UNITY_ERR_INVALID_ARG, "logp_in, entropy_in and lse_in must be given together");

    // choose gradient chunk sizes that fit the workspace
    int cr = wanted_chunk_rows(rows->n_tok, K, ctx->chunk_rows_mult), cv = wanted_chunk_vocab(V, ctx->chunk_vocab_mult);
    RowPlan P;
    bool fits = false;
    // Logit stash: the forward runs block by block of rows and keeps the block's scaled logits (bf16, one slab per
    // vocabulary chunk); the backward turns each slab into dL/dz in place instead of recomputing the logits.
    bool stash = ctx->logit_stash && !have_fwd;
    int z_base = 0, z_chunks = 0;
    if (stash) {
        const int cr_s = cr < kStashRows ? cr : kStashRows, cv_s = wanted_chunk_vocab(V, ctx->chunk_vocab_mult);
        vocab_chunks(V, cv_s, &z_base, &z_chunks);
        P.L = carve(ctx->ws, ctx->ws_bytes, rows->n_tok, H, V, K, rows->n_inv, cr_s, cv_s, &fits, z_chunks);
        if (fits) { cr = cr_s; cv = cv_s; }
        else stash = false;                     // workspace without room for the stash: recompute instead
    }
    while (!stash) {
        P.L = carve(ctx->ws, ctx->ws_bytes, rows->n_tok, H, V, K, rows->n_inv, cr, cv, &fits);
        if (fits) break;
        if (cr > kMinChunkRows && cr >= cv) cr = static_cast<int>(up(cr / 2, kTileM));
        else if (cv > kMinChunkVocab) cv = static_cast<int>(up(cv / 2, kTileN));
        else if (cr > kMinChunkRows) cr = static_cast<int>(up(cr / 2, kTileM));
        else return fail(ctx, UNITY_ERR_WORKSPACE, "workspace too small: need at least %zu bytes, have %zu", P.L.bytes, ctx->ws_bytes);
    }
    const Layout& L = P.L;

    CUDA_TRY(ctx, cudaMemsetAsync(loss, 0, sizeof(float) * K, st));
    if (rows->n_tok == 0) {
        if (metrics) CUDA_TRY(ctx, cudaMemsetAsync(metrics, 0, sizeof(float) * (K + rows->n_roles) * UNITY_N_METRICS, st));
        if (!params->accumulate_dW)
            for (int k = 0; k < K; ++k) CUDA_TRY(ctx, cudaMemsetAsync(dW[k], 0, sizeof(float) * V * H, st));
        return UNITY_OK;
    }
    if (logp) CUDA_TRY(ctx, cudaMemsetAsync(logp, 0, sizeof(float) * rows->n_tok, st));
    if (entropy) CUDA_TRY(ctx, cudaMemsetAsync(entropy, 0, sizeof(float) * rows->n_tok, st));
    if (tok_loss) CUDA_TRY(ctx, cudaMemsetAsync(tok_loss, 0, sizeof(float) * rows->n_tok, st));

    rc = forward_sweep(ctx, rows, P, !have_fwd && !stash);
    if (rc) return rc;
    int nl = 0;

    TokenArgs t;
    fill_token_args(t, rows, P);
    t.logp = logp; t.entropy = entropy; t.lse = nullptr;
    if (have_fwd) { t.logp_in = params->logp_in; t.entropy_in = params->entropy_in; t.lse_in = params->lse_in; }
    t.old_logp = old_logp; t.ref_logp = ref_logp; t.adv_tok = adv_tok;
    t.clip_lo = params->clip_lo; t.clip_hi = params->clip_hi; t.kl_coef = params->kl_coef;
    t.ent_coef = params->ent_coef; t.kl_mode = params->kl_mode;
    t.has_norm = params->norm != nullptr;
    for (int k = 0; k < K && params->norm; ++k) t.norm[k] = params->norm[k];
    t.coef_a = L.coef_a; t.coef_b = L.coef_b; t.tok_loss = tok_loss;
    t.inv_sums = L.inv_sums; t.loss = loss; t.metrics = metrics;
    if (!stash) CUDA_TRY(ctx, launch_finish_forward(t, true, st, &nl));

    __nv_bfloat16* dH = static_cast<__nv_bfloat16*>(dHidden);
    CUDA_TRY(ctx, launch_zero_masked_rows(L.tok_slot, rows->n_tok, H, dH, st));
    nl += 1;
    // Operands are read in place: hidden rows and W serve as K-major operands (contraction over H) and as
    // MN-major operands (contraction over tokens / vocabulary); nothing is transposed in memory.
    CUtensorMap tm_hp_k, tm_hp_mn;
    if ((rc = make_tmap(ctx, &tm_hp_k, L.hp, H, L.max_slots, static_cast<uint64_t>(H) * 2, kBoxRows))) return rc;
    if ((rc = make_tmap(ctx, &tm_hp_mn, L.hp, H, L.max_slots, static_cast<uint64_t>(H) * 2, kTileK))) return rc;
    // Tiles two blocks wide unless one-block tiles waste clearly less of this launch: the share of executed MMA work that
    // is useful = (H / padded columns) x (tiles / tiles rounded up to whole waves of CTA pairs); the wide form gets a
    // 15 % bonus for its lower operand traffic (at H = 896 the narrow form is bound by the stream of G, not by MMA time:
    // dHidden +13 %, dW +7 % with the wide form although it wastes an eighth more of its last wave).
    const int n_workers = ctx->sm_count / 2;
    auto pick_wide = [&](int cls, int m_tiles) {
        if (!ctx->wide_acc || ctx->ctas[cls] != 2) return false;
        const int mma_n = gemm_mma_n(H);
        auto useful = [&](int blocks) {
            const int cols = blocks * mma_n;
            const long long nt = (H + cols - 1) / cols, tiles = nt * m_tiles;
            const long long waves = (tiles + n_workers - 1) / n_workers;
            return (static_cast<double>(H) / (nt * cols)) * (static_cast<double>(tiles) / (waves * n_workers));
        };
        return m_tiles <= 0 || 1.15 * useful(2) >= useful(1);
    };
    const int c_grad = ctx->ctas[UNITY_PROF_GRAD_GEMM], c_dh = ctx->ctas[UNITY_PROF_DH_GEMM],
              c_dw = ctx->ctas[UNITY_PROF_DW_GEMM];

    // The host does not know how many rows a model has (unless it was asked to read the counts back): it walks every
    // chunk a model could have, each kernel cuts its span to the rows that exist, and a launch without rows returns at once.
    for (int k = 0; k < K; ++k) {
        const long long rows_k = rows_of(P, k);
        float* dWk = static_cast<float*>(dW[k]);
        // nothing accumulates into the dW of a model without rows: it must still read zero
        if (!params->accumulate_dW) {
            if (rows_k == 0) CUDA_TRY(ctx, cudaMemsetAsync(dWk, 0, sizeof(float) * V * H, st));
            else if (P.rows_known[k] < 0) { CUDA_TRY(ctx, launch_zero_if_empty(dWk, static_cast<long long>(V) * H, L.plan, k, st)); nl += 1; }
        }
        if (rows_k == 0) continue;
        const __nv_bfloat16* Wk = static_cast<const __nv_bfloat16*>(rows->W[k]);
        CUtensorMap tm_W_k, tm_W_mn, tm_W_f;
        if ((rc = make_tmap(ctx, &tm_W_k, Wk, H, V, static_cast<uint64_t>(H) * 2, kTileN / c_grad))) return rc;
        if (stash && (rc = make_tmap(ctx, &tm_W_f, Wk, H, V, static_cast<uint64_t>(H) * 2, kTileN / ctx->ctas[UNITY_PROF_FWD_GEMM]))) return rc;
        if ((rc = make_tmap(ctx, &tm_W_mn, Wk, H, V, static_cast<uint64_t>(H) * 2, kTileK))) return rc;

        for (long long c0 = 0; c0 < rows_k; c0 += cr) {
            const int nc = static_cast<int>(rows_k - c0 < cr ? rows_k - c0 : cr);   // at most this many rows (multiple of kTileM)
            const RowSpan chunk{L.plan, k, static_cast<int>(c0), nc};
            if (stash) {
                // forward over this block of rows, keeping its logits; then the per-row loss terms of the block
                const ZStash z{L.G, cv, static_cast<long long>(cr) * cv, z_base, z_chunks};
                if ((rc = launch_forward(ctx, rows, P, chunk, false, tm_hp_k, tm_W_f, &z))) return rc;
                TokenArgs tc = t;
                tc.block = chunk;
                CUDA_TRY(ctx, launch_finish_rows(tc, true, st, &nl));
                nl += 1;
            }
            const int tail = kTailTiles * kTileN;
            const int base = (V > cv && cv > tail + kTileN) ? cv - tail : cv;      // regular chunk width
            int ci = 0;
            for (int v0 = 0, vc = 0; v0 < V; v0 += vc, ++ci) {
                vc = V - v0 < base ? V - v0 : base;
                if (V - (v0 + vc) <= tail && base < cv) vc = V - v0;               // absorb a short remainder
                __nv_bfloat16* Gc = stash ? L.G + static_cast<long long>(ci) * cr * cv : L.G;
                // (1) dL/dz of this (rows x vocab) chunk in bf16: G[nc, vc]
                if (stash) {
                    LogitGradArgs lg;
                    memset(&lg, 0, sizeof(lg));
                    lg.Z = Gc; lg.ld = cv; lg.span = chunk; lg.cols = vc; lg.vocab0 = v0;
                    lg.target_p = L.target_p; lg.coef_a = L.coef_a; lg.coef_b = L.coef_b;
                    lg.row_lse = L.row_lse; lg.row_ent = L.row_ent;
                    ProfScope ps(ctx, UNITY_PROF_GRAD_GEMM);
                    CUDA_TRY(ctx, launch_logit_grad_inplace(lg, st));
                    nl += 1;
                } else {
                    // recompute the logits.  Whatever the chunk size, one launch covers at most kChunkRows x
                    // (kChunkVocab + tail) of it: the kernel re-reads its W block once per group of row tiles, and
                    // that block has to stay small enough for the group's hidden rows to survive in L2 meanwhile.
                    // (On the forward's schedule a round bounds the rows in flight by itself and a launch may cover more.)
                    const int rounds = ctx->grad_rounds >= 0 ? ctx->grad_rounds : (large_rounds_fit(ctx, H) ? ctx->sm_count / 2 : 0);
                    int runs = rounds > 0 ? 0 : ctx->grad_runs;
                    if (runs < 0) {   // 128-row tiles whose hidden rows fit the 45 MB share of L2
                        runs = static_cast<int>((45ll << 20) / (128ll * H * 2));
                        runs = runs < 8 ? 8 : (runs > ctx->sm_count / 2 ? ctx->sm_count / 2 : runs);
                    }
                    const int per_side = ctx->grad_block > 0 ? ctx->grad_block : (rounds > 0 || runs > 0 ? 8 : 1);
                    const int blk_rows = kChunkRows * per_side, blk_cols = kChunkVocab * per_side;
                    for (int r0 = 0; r0 < nc; r0 += blk_rows) {
                        const int nr = nc - r0 < blk_rows ? nc - r0 : blk_rows;
                        for (int q0 = 0, qc = 0; q0 < vc; q0 += qc) {
                            qc = vc - q0 < blk_cols ? vc - q0 : blk_cols;
                            if (vc - (q0 + qc) <= tail) qc = vc - q0;
                            GemmArgs g;
                            memset(&g, 0, sizeof(g));
                            g.span = RowSpan{L.plan, k, static_cast<int>(c0) + r0, nr}; g.span_mode = kSpanRowsA;
                            g.m_tiles = 1;                                   // set by the kernel
                            g.n_tiles = (qc + kTileN - 1) / kTileN; g.k_iters = H / kTileK;
                            g.group_m = ctx->chunk_group[0] / c_grad > 0 ? ctx->chunk_group[0] / c_grad : 1;
                            if (runs > 0) {
                                g.plan_runs = 1;
                                g.fwd.n_pairs = ctx->sm_count / c_grad;
                                g.fwd.tile_rows = gemm_tile_rows(c_grad);
                                g.fwd.n_tiles = g.n_tiles;
                                g.fwd.gmax = runs / c_grad > 0 ? runs / c_grad : 1;
                            }
                            if (rounds > 0) {
                                g.fwd.n_pairs = ctx->sm_count / c_grad;
                                g.fwd.tile_rows = gemm_tile_rows(c_grad);
                                g.fwd.n_tiles = g.n_tiles;
                                g.fwd.gmax = rounds / c_grad > 0 ? rounds / c_grad : 1;
                                if (g.fwd.gmax > g.fwd.n_pairs) g.fwd.gmax = g.fwd.n_pairs;
                            }
                            g.a_row0 = 0; g.b_row0 = v0 + q0; g.n_cols = qc;
                            g.target_p = L.target_p; g.vocab0 = v0 + q0; g.scale = rows->inv_temperature;
                            g.coef_a = L.coef_a; g.coef_b = L.coef_b; g.row_lse = L.row_lse; g.row_ent = L.row_ent;
                            g.has_ent = params->ent_coef != 0.f;
                            g.G = Gc + static_cast<long long>(r0) * cv + q0; g.ldg = cv;
                            g.g_wide_store = (reinterpret_cast<uintptr_t>(g.G) % 32 == 0) && (g.ldg * 2 % 32 == 0);
                            gemm_common(ctx, g, UNITY_PROF_GRAD_GEMM, &P.counters, (ctx->chunk_sync & 1) != 0);
                            ProfScope ps(ctx, UNITY_PROF_GRAD_GEMM);
                            CUDA_TRY(ctx, launch_gemm(kEpiLogitGrad, false, c_grad, tm_hp_k, tm_W_k, g, ctx->sm_count, st));
                            nl += 1;
                        }
                    }
                }
                // G viewed as [rows, vc]: K-major A for dHidden (contract over vc), MN-major A for dW (rows = K)
                CUtensorMap tm_G_k, tm_G_mn;
                if ((rc = make_tmap(ctx, &tm_G_k, Gc, vc, nc, static_cast<uint64_t>(cv) * 2, kBoxRows))) return rc;
                if ((rc = make_tmap(ctx, &tm_G_mn, Gc, vc, nc, static_cast<uint64_t>(cv) * 2, kTileK))) return rc;
                // (2) dH_chunk[rows, H] (+)= G[rows, vc] * W[v0:v0+vc, :]      (B = W, MN-major: rows v are K)
                GemmArgs h;
                memset(&h, 0, sizeof(h));
                const bool wide_dh = pick_wide(UNITY_PROF_DH_GEMM, nc / gemm_tile_rows(c_dh));
                const int mma_n = gemm_mma_n(H);                       // dHidden and dW both have H output columns
                const int cols_dh = (wide_dh ? 2 : 1) * mma_n;
                h.mma_n = mma_n;
                h.span = chunk; h.span_mode = kSpanRowsM;
                h.m_tiles = 1;                                         // set by the kernel
                h.n_tiles = (H + cols_dh - 1) / cols_dh;
                h.k_iters = (vc + kTileK - 1) / kTileK;
                h.group_m = ctx->chunk_group[1] / c_dh > 0 ? ctx->chunk_group[1] / c_dh : 1;
                h.a_row0 = 0; h.a_k0 = 0; h.b_row0 = 0; h.b_k0 = v0; h.n_cols = H;
                h.C = L.dHc; h.ldc = H; h.beta = v0 > 0;
                gemm_common(ctx, h, UNITY_PROF_DH_GEMM, &P.counters, (ctx->chunk_sync & 2) != 0);
                {
                    ProfScope ps(ctx, UNITY_PROF_DH_GEMM);
                    CUDA_TRY(ctx, launch_gemm(kEpiAccumF32, false, c_dh, tm_G_k, tm_W_mn, h, ctx->sm_count, st, wide_dh));
                }
                // (3) dW[v0:v0+vc, :] (+)= G^T[vc, rows] * hidden[first slot of the chunk ..., :]   (both operands MN-major)
                // The vocabulary tiles of a chunk are known here.  When the last few of them would open one more wave of
                // workers and fill less than half of it (V = 152064: a last chunk of 150 tiles after three of 148), they run
                // as a launch of their own with narrow tiles, so that they spread over the machine instead of occupying a
                // seventh of it for a whole tile time.
                const int tile_v = gemm_tile_rows(c_dw), vt = (vc + tile_v - 1) / tile_v;
                const bool wide_all = pick_wide(UNITY_PROF_DW_GEMM, vt);
                int vt_main = vt, narrow_n = 0;
                if (ctx->dw_tail && c_dw == 2 && vt > n_workers) {
                    const int nt_main = (H + (wide_all ? 2 : 1) * mma_n - 1) / ((wide_all ? 2 : 1) * mma_n);
                    const int rem = vt % n_workers;
                    if (rem > 0 && 2 * rem * nt_main < n_workers) {
                        for (int cand = 64; cand <= kTileN && narrow_n == 0; cand += 32)
                            if (static_cast<long long>(rem) * ((H + cand - 1) / cand) <= n_workers) narrow_n = cand;
                        if (narrow_n > 0) vt_main = vt - rem;
                    }
                }
                for (int part = 0; part < (narrow_n > 0 ? 2 : 1); ++part) {
                    const int t0 = part == 0 ? 0 : vt_main, t1 = part == 0 ? vt_main : vt;
                    const int row0 = t0 * tile_v, rows_here = (t1 * tile_v < vc ? t1 * tile_v : vc) - row0;
                    GemmArgs w;
                    memset(&w, 0, sizeof(w));
                    w.m_tiles = t1 - t0;
                    const bool wide_dw = part == 0 && pick_wide(UNITY_PROF_DW_GEMM, w.m_tiles);
                    w.mma_n = part == 0 ? mma_n : narrow_n;
                    const int cols_dw = (wide_dw ? 2 : 1) * w.mma_n;
                    w.span = chunk; w.span_mode = kSpanRowsK;
                    w.n_tiles = (H + cols_dw - 1) / cols_dw;
                    w.k_iters = 1;                                         // set by the kernel
                    w.group_m = ctx->chunk_group[2] / c_dw > 0 ? ctx->chunk_group[2] / c_dw : 1;
                    w.a_row0 = row0; w.a_k0 = 0; w.b_row0 = 0; w.b_k0 = 0; w.m_rows = rows_here; w.n_cols = H;
                    w.C = dWk + static_cast<long long>(v0 + row0) * H; w.ldc = H;
                    w.beta = (params->accumulate_dW || c0 > 0) ? 1 : 0;
                    gemm_common(ctx, w, UNITY_PROF_DW_GEMM, &P.counters, (ctx->chunk_sync & 4) != 0);
                    ProfScope ps(ctx, UNITY_PROF_DW_GEMM);
                    CUDA_TRY(ctx, launch_gemm(kEpiAccumF32, true, c_dw, tm_G_mn, tm_hp_mn, w, ctx->sm_count, st, wide_dw));
                    nl += 1;
                }
                nl += 1;
            }
            CUDA_TRY(ctx, launch_store_dhidden(L.dHc, L.slot_tok, chunk, H, dH, st));
            nl += 1;
        }
    }
    if (stash) CUDA_TRY(ctx, launch_loss_reduce(t, st, &nl));
    ctx->launches += nl;
    return UNITY_OK;
}

}  // extern "C"
