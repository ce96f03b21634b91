// Persistent, warp-specialised bf16 GEMM for sm_100a:  C[m, n] = sum_k A[m, k] * B[n, k], each operand either
// K-major ([rows, K] in memory) or MN-major ([K, rows] in memory), so no operand is ever transposed in HBM.
//
// The kernel exists in two forms (template parameter CTAS):
//   CTAS = 1 : one CTA computes a 128 x 256 output tile (tcgen05.mma.cta_group::1), 4-stage ring of 48 KiB slabs.
//   CTAS = 2 : two CTAs on neighbouring SMs (a cluster of 2) share one 256 x 256 tile: each loads its own 128 rows
//              of A and its own 128 of the 256 rows of B (32 KiB per K slab, 7-stage ring) and one
//              tcgen05.mma.cta_group::2 issued by the even CTA multiplies across both shared memories; each CTA's
//              tensor memory receives the 128 x 256 accumulator block of its own rows.
// Per CTA:
//   warp 0      : TMA producer  - streams its A and B slabs into the shared-memory ring; with CTAS = 2 the bytes of
//                                 both CTAs are counted on the even CTA's barrier
//   warp 1      : MMA issuer    - one thread (of the even CTA) issues the MMAs into one of two 256-column
//                                 accumulator stages and commits completion to the barriers of the CTA(s)
//   warps 2..5  : epilogue      - each thread owns one accumulator row (one TMEM lane), drains it 32 columns at a
//                                 time with tcgen05.ld while the MMAs already fill the other stage
//
// The fp32-accumulate epilogue also exists with tiles two MMA blocks wide (template parameter NB = 2, CTA pairs
// only): two MMAs per K step fill all of tensor memory as ONE accumulator stage, so a K slab of A is loaded once for
// twice the columns (a quarter less operand traffic from L2 and DRAM).  The epilogue then does not overlap the next
// tile's MMAs, which is affordable only because these GEMMs contract over a whole gradient chunk (hundreds of K
// slabs per tile); it adds into C with fire-and-forget vector reductions instead of load-add-store.  The block width of
// this epilogue is a run-time value (GemmArgs::mma_n, a multiple of 32 up to 256): an output of 896 columns runs as
// blocks of 224 instead of padding a fourth block of 256 with zeros.
//
// Three epilogues share the main loop:
//   softmax statistics : running (max, sum exp, sum exp*z, target logit) per row across a sweep of vocabulary
//                        tiles; nothing of size rows x vocabulary is ever written
//   logit gradient     : dL/dz = a*(onehot - p) - b*p*(z - lse + H) in bf16 for a bounded chunk
//   fp32 accumulate    : C (+)= acc
// Every mbarrier wait is bounded; on expiry the CTA records a timeout status, all its roles leave their loops, and
// after a cluster-wide rendezvous the CTA(s) free their tensor memory and return.
#include <cstring>

#include "internal.h"
#include "ptx.cuh"

namespace unity {

namespace {

constexpr int kTmemCols = 2 * kTileN;                     // 512: all of tensor memory (two stages of 256 or one of 512)
constexpr int kBarBytes = 256;
constexpr int kThreads = 192;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegBig = -3.0e38f;
// MN-major operands: a stage holds boxes of 64 rows x 64 K (8 KiB), one after the other.
constexpr int kMnBoxBytes = 64 * kTileK * 2;

template <int CTAS, int NB = 1>
struct Cfg {
    static constexpr int kTileRows = kCtaM * CTAS;               // rows of one output tile (128 or 256)
    static constexpr int kTileCols = kTileN * NB;                // columns of one output tile (256 or 512)
    static constexpr int kAccStages = 2 / NB;                    // accumulator stages in tensor memory
    static constexpr int kBRows = kTileN / CTAS;                 // rows of B this CTA loads per 256-column block
    static constexpr int kABytes = kCtaM * kTileK * 2;           // 16 KiB
    static constexpr int kBBytes = kBRows * kTileK * 2;          // 32 or 16 KiB per 256-column block
    static constexpr int kStageBytes = kABytes + NB * kBBytes;   // 48 or 32 KiB
    static constexpr int kStages = (CTAS == 1 || NB == 2) ? 4 : 7;
    static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kBarBytes;
};

struct Unit {
    int m_tile, n_begin, n_end, split;
    bool rev;     // walk the unit's column tiles from n_end - 1 down to n_begin
};

// Column tiles per unit of the striding schedule (below): one, or a run of GemmArgs::unit_tiles (logit gradient only).
template <int EPI>
__device__ __forceinline__ int stride_unit_tiles(const GemmArgs& g) {
    return EPI == kEpiLogitGrad && g.unit_tiles > 1 ? g.unit_tiles : 1;
}
// The logit-gradient epilogue can run on the softmax epilogue's schedule of rounds: the launch says so by carrying a
// split count.
template <int EPI>
__device__ __forceinline__ bool in_rounds(const GemmArgs& g) {
    return EPI == kEpiSoftmaxStats || (EPI == kEpiLogitGrad && g.n_splits > 0);
}

// Work decomposition over workers (CTAs or CTA pairs); `it` counts the iterations of a worker's persistent loop.
// Rounds (softmax statistics always; logit gradient when the launch carries a split count): a unit is (row tile,
// vocabulary split).  Round `it` works on row-tile group `it` (gm row tiles): worker p takes split p / gm_here of row
// tile p % gm_here and workers beyond gm_here * n_splits sit the round out.  All workers of a round therefore share gm
// A tiles (L2 resident) and each split's stream of B tiles is fetched from HBM once, by workers that sweep it in step.
// Striding (the other launches): unit = worker + it * workers, m fastest inside groups of gm row tiles; a unit is one
// output tile, with the column order alternating from one group of row tiles to the next, or a run of column tiles.
// Returns false when the worker has no more work; `valid` is false for a round the worker sits out.
template <int EPI>
__device__ __forceinline__ bool next_unit(const GemmArgs& g, int it, int pair, int n_pairs, int gm, Unit& t, bool& valid) {
    t.rev = false;
    if (in_rounds<EPI>(g)) {
        const int m0 = it * gm;
        if (m0 >= g.m_tiles) return false;
        const int gm_here = min(gm, g.m_tiles - m0);
        const bool last = m0 >= g.last_m0;                       // the short last round: more, shorter splits
        const int n_splits = last ? g.last_splits : g.n_splits;
        const int tps = last ? g.last_tiles_per_split : g.tiles_per_split;
        valid = pair < gm_here * n_splits;
        t.split = pair / gm_here;
        t.m_tile = m0 + (pair - t.split * gm_here);
        t.n_begin = t.split * tps;
        t.n_end = min(t.n_begin + tps, g.n_tiles);
        // logit gradient: odd rounds sweep their split backwards, so a round starts on the W tiles the round before it
        // ended with (the statistics of the softmax epilogue depend on the order of the sweep and keep it)
        t.rev = EPI == kEpiLogitGrad && (it & 1);
        return true;
    } else {
        // a unit is one output tile, or (logit gradient, GemmArgs::unit_tiles > 1) a run of that many column tiles of one
        // row tile: all units of a launch are then nearly equally long, every worker holds one at any time, and the
        // workers that hold the same run of columns sweep its W tiles in step
        const int tpu = stride_unit_tiles<EPI>(g);
        const int ncu = (g.n_tiles + tpu - 1) / tpu;
        const int u = pair + it * n_pairs;
        if (u >= g.m_tiles * ncu) return false;
        const int per_group = gm * ncu;
        const int grp = u / per_group, r = u - grp * per_group;
        const int m0 = grp * gm;
        const int gm_here = min(gm, g.m_tiles - m0);
        const int q = r / gm_here;
        t.m_tile = m0 + (r - q * gm_here);
        t.split = 0;
        if (tpu == 1) {
            // odd groups walk the columns backwards: the B tiles a group ends with are the ones the next group starts
            // with, while they are still in L2
            t.n_begin = (grp & 1) ? g.n_tiles - 1 - q : q;
            t.n_end = t.n_begin + 1;
        } else {
            t.n_begin = q * tpu;
            t.n_end = min(t.n_begin + tpu, g.n_tiles);
        }
        valid = true;
        return true;
    }
}

__device__ __forceinline__ unsigned pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<unsigned*>(&v);
}

// The launch's arguments with everything that depends on the number of rows filled in from the device plan.
template <int TILE_ROWS>
__device__ __noinline__ GemmArgs resolve_span(const GemmArgs& in) {
    GemmArgs g = in;
    if (in.span.plan == nullptr) return g;
    int slot0, n_rows;
    span_resolve(in.span, slot0, n_rows);
    if (in.span_mode == kSpanForward) {
        const FwdShape fs = forward_shape(in.fwd, n_rows);
        g.a_row0 = slot0;
        g.m_rows = n_rows;
        g.m_tiles = n_rows / TILE_ROWS;
        g.group_m = fs.gm; g.n_splits = fs.splits; g.tiles_per_split = fs.tps;
        g.last_m0 = fs.last_m0; g.last_splits = fs.last_splits; g.last_tiles_per_split = fs.last_tps;
        g.last_stats_off = static_cast<long long>(fs.splits) * n_rows;
        g.last_pitch = n_rows - static_cast<long long>(fs.last_m0) * TILE_ROWS;
        g.stats_pitch = n_rows;
        {   // the most units any round holds: a full round, or the short last one with its own split count
            const int full = min(g.m_tiles, fs.gm) * fs.splits, last = (g.m_tiles - fs.last_m0) * fs.last_splits;
            g.n_active = max(full, last);
        }
        if (in.stats_from_plan) g.stats = in.stats + in.span.plan->stats_base[in.span.model];
    } else if (in.span_mode == kSpanRowsA) {
        g.a_row0 = in.a_row0 + slot0;
        g.m_rows = n_rows;
        g.m_tiles = n_rows / TILE_ROWS;
        if (in.fwd.n_pairs > 0 && in.plan_runs) {
            // Units = runs of column tiles.  More runs than the L2 budget asks for (fwd.gmax row tiles in flight) are
            // fine; among a few counts take the one whose units fill the workers' iterations best.
            const int np = in.fwd.n_pairs, nt = in.n_tiles;
            const int ncu_min = max(1, (np + in.fwd.gmax - 1) / in.fwd.gmax);
            int best_tpu = nt, best_ncu = 1;
            long long best_cost = -1;
            for (int want = ncu_min; want <= min(nt, ncu_min + 12); ++want) {
                const int tpu = (nt + want - 1) / want, ncu = (nt + tpu - 1) / tpu;
                const long long cost = (static_cast<long long>(g.m_tiles) * ncu + np - 1) / np * tpu;
                if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_tpu = tpu; best_ncu = ncu; }
            }
            g.unit_tiles = best_tpu;
            g.group_m = max(1, min(g.m_tiles, (np + best_ncu - 1) / best_ncu));
            const long long units = static_cast<long long>(g.m_tiles) * best_ncu;
            g.n_active = static_cast<int>(min(static_cast<long long>(np), units));
        } else if (in.fwd.n_pairs > 0) {
            // the recompute GEMM on the forward's schedule: rounds of row tiles x vocabulary splits of this launch's columns
            const FwdShape fs = forward_shape(in.fwd, n_rows);
            g.group_m = fs.gm; g.n_splits = fs.splits; g.tiles_per_split = fs.tps;
            g.last_m0 = fs.last_m0; g.last_splits = fs.last_splits; g.last_tiles_per_split = fs.last_tps;
            const int full = min(g.m_tiles, fs.gm) * fs.splits, last = (g.m_tiles - fs.last_m0) * fs.last_splits;
            g.n_active = max(full, last);
        }
    } else if (in.span_mode == kSpanRowsM) {
        g.m_rows = n_rows;
        g.m_tiles = n_rows / TILE_ROWS;
    } else if (in.span_mode == kSpanRowsK) {
        g.k_iters = n_rows / kTileK;
        g.b_k0 = in.b_k0 + slot0;
    }
    return g;
}

template <int EPI, bool A_MN, bool B_MN, int CTAS, int NB = 1>
__global__ void __launch_bounds__(kThreads, 1)
k_gemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmArgs g_in) {
    using C = Cfg<CTAS, NB>;
    // The row extent of a launch may be known on the device only: derive it from the plan before anything else.  Every
    // thread of both CTAs reads the same plan, so a launch whose span is empty is left by all of them, here.
    const GemmArgs g = resolve_span<C::kTileRows>(g_in);
    if (g.m_tiles <= 0 || g.n_tiles <= 0 || g.k_iters <= 0) return;
    if (g.n_active > 0 && (CTAS == 2 ? blockIdx.x >> 1 : blockIdx.x) >= g.n_active) return;   // never holds a unit
    constexpr int kStages = C::kStages, kStageBytes = C::kStageBytes, kABytes = C::kABytes, kBBytes = C::kBBytes;
    constexpr int kAccStages = C::kAccStages, kTileCols = C::kTileCols;
    static_assert(NB == 1 || (EPI == kEpiAccumF32 && CTAS == 2), "two-block tiles: fp32-accumulate epilogue, CTA pairs");
    extern __shared__ uint8_t smem_raw[];
    // the dynamic shared-memory window starts at the same offset in both CTAs of a pair, so all offsets below match
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
    uint64_t* full = bars;                       // [kStages]  (even CTA) bytes of both CTAs landed
    uint64_t* empty = bars + kStages;            // [kStages]  MMAs that read the stage have completed
    uint64_t* acc_full = bars + 2 * kStages;     // [2]        accumulator stage complete
    uint64_t* acc_empty = acc_full + kAccStages; // [2]        (even CTA) stage drained by the epilogues of both CTAs
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + kAccStages);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta_rank = CTAS == 2 ? ptx::cluster_ctarank() : 0u;     // 0: issues the MMAs, 1: its peer
    const int pair = CTAS == 2 ? blockIdx.x >> 1 : blockIdx.x;              // index of this worker (CTA or CTA pair)
    const int n_launched = CTAS == 2 ? gridDim.x >> 1 : gridDim.x;
    const int n_pairs = g.n_active > 0 && g.n_active < n_launched ? g.n_active : n_launched;   // workers at work

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
        for (int s = 0; s < kAccStages; ++s) { ptx::mbar_init(&acc_full[s], 1); ptx::mbar_init(&acc_empty[s], 4 * CTAS); }
        *abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmB);
    }
    if (warp == 1) {
        if (CTAS == 2) { ptx::tmem_alloc_pair(tmem_slot, kTmemCols); ptx::tmem_relinquish_pair(); }
        else { ptx::tmem_alloc(tmem_slot, kTmemCols); ptx::tmem_relinquish(); }
    }
    ptx::tc_fence_before();
    if (CTAS == 2) ptx::cluster_sync_all();   // barriers of both CTAs are initialised before anyone signals across
    else __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int gm = max(1, g.group_m);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            const uint64_t pol_a = ptx::l2_policy(g.l2_hints & 3), pol_b = ptx::l2_policy((g.l2_hints >> 2) & 3);
            for (int it = 0; ok; ++it) {
                Unit t;
                bool valid;
                if (!next_unit<EPI>(g, it, pair, n_pairs, gm, t, valid)) break;
                if (g.round_counter != nullptr && cta_rank == 0 && (in_rounds<EPI>(g) || it % g.sync_period == 0)) {
                    // Soft rendezvous at the start of a round (softmax: every round; other epilogues, whose round is one
                    // tile: every sync_period-th): the workers that share a stream of W tiles stay in step only while
                    // they start together, and once they drift apart by more than L2 can bridge each of them fetches the
                    // stream from HBM again.  Purely a performance hint: after a short, bounded wait the worker goes on
                    // regardless (some CTAs may not be resident yet).
                    // The counter belongs to this launch and starts at zero.
                    atomicAdd(g.round_counter, 1u);
                    // arrivals expected by the end of this rendezvous: every worker (softmax), or every worker that
                    // still has a tile (the last ones of the other epilogues may be partial)
                    unsigned expect;
                    if (in_rounds<EPI>(g)) {
                        expect = static_cast<unsigned>(it + 1) * static_cast<unsigned>(n_pairs);
                    } else {
                        const long long before = static_cast<long long>(it) * n_pairs;      // units of earlier rounds
                        const int tpu = stride_unit_tiles<EPI>(g);
                        const long long left = static_cast<long long>(g.m_tiles) * ((g.n_tiles + tpu - 1) / tpu) - before;
                        expect = static_cast<unsigned>(it / g.sync_period) * static_cast<unsigned>(n_pairs) +
                                 static_cast<unsigned>(left < n_pairs ? left : n_pairs);
                    }
                    const unsigned target = expect;
                    const long long t0 = clock64();
                    while (static_cast<int>(*reinterpret_cast<volatile unsigned*>(g.round_counter) - target) < 0 &&
                           clock64() - t0 < 400000) { }
                }
                if (!valid) continue;
                const int a_row = g.a_row0 + t.m_tile * C::kTileRows + static_cast<int>(cta_rank) * kCtaM;
                for (int ni = t.n_begin; ni < t.n_end && ok; ++ni) {
                    const int nt = t.rev ? t.n_begin + t.n_end - 1 - ni : ni;
                    // fp32-accumulate tiles may be narrower than 256 columns per MMA (mma_n); the B boxes keep their size, the
                    // MMA simply leaves their last columns unread
                    const int mma_n = EPI == kEpiAccumF32 ? g.mma_n : kTileN;
                    const int b_row = g.b_row0 + nt * (NB * mma_n) + static_cast<int>(cta_rank) * (mma_n / CTAS);
                    for (int k = 0; k < g.k_iters; ++k) {
                        if (!ptx::mbar_wait(&empty[stage], phase ^ 1, g.wait_budget) || *abort_flag) { ok = false; break; }
                        if (g.test_drop_slab && it == 0 && ni == t.n_begin && k == (g.k_iters > 1 ? 1 : 0)) {
                            // test hook: this slab never arrives; the MMA issuer's wait for it must run out
                            if (++stage == kStages) { stage = 0; phase ^= 1; }
                            continue;
                        }
                        uint8_t* sA = smem + stage * kStageBytes;
                        // completion bytes are counted on the barrier of the CTA that issues the MMAs
                        const uint32_t bar = CTAS == 2 ? ptx::mapa(ptx::smem_u32(&full[stage]), 0) : ptx::smem_u32(&full[stage]);
                        if (cta_rank == 0) ptx::mbar_arrive_expect_tx(&full[stage], CTAS * kStageBytes);
                        if (A_MN) {
#pragma unroll
                            for (int j = 0; j < kCtaM / 64; ++j)
                                ptx::tma_load_2d_hint_on<CTAS>(sA + j * kMnBoxBytes, &tmA, bar, a_row + j * 64, g.a_k0 + k * kTileK, pol_a);
                        } else {
                            ptx::tma_load_2d_hint_on<CTAS>(sA, &tmA, bar, g.a_k0 + k * kTileK, a_row, pol_a);
                        }
#pragma unroll
                        for (int nb = 0; nb < NB; ++nb) {          // one block of B rows per 256 output columns
                            uint8_t* sB = sA + kABytes + nb * kBBytes;
                            if (B_MN) {
#pragma unroll
                                for (int j = 0; j < C::kBRows / 64; ++j)
                                    ptx::tma_load_2d_hint_on<CTAS>(sB + j * kMnBoxBytes, &tmB, bar, b_row + nb * mma_n + j * 64,
                                                                   g.b_k0 + k * kTileK, pol_b);
                            } else {
                                ptx::tma_load_2d_hint_on<CTAS>(sB, &tmB, bar, g.b_k0 + k * kTileK, b_row + nb * mma_n, pol_b);
                            }
                        }
                        if (++stage == kStages) { stage = 0; phase ^= 1; }
                    }
                }
            }
            if (!ok) { *abort_flag = 1; atomicOr(g.status, kStatusTimeout); }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (even CTA only)
        if (lane == 0 && cta_rank == 0) {
            const uint32_t idesc = ptx::idesc_bf16_f32(C::kTileRows, EPI == kEpiAccumF32 ? g.mma_n : kTileN) |
                                   (A_MN ? (1u << 15) : 0u) | (B_MN ? (1u << 16) : 0u);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            // `ready` is the answer of a non-blocking look at full[stage], issued one step earlier (before that step's
            // MMAs): a barrier query between two groups of MMAs otherwise leaves the tensor pipe idle for its latency
            // (measured: 135 instead of 128 clocks per MMA).
            bool ready = false;
            for (int it = 0; ok; ++it) {
                Unit t;
                bool valid;
                if (!next_unit<EPI>(g, it, pair, n_pairs, gm, t, valid)) break;
                if (!valid) continue;
                for (int nt = t.n_begin; nt < t.n_end && ok; ++nt) {
                    if (!ptx::mbar_wait(&acc_empty[acc], acc_phase ^ 1, g.wait_budget) || *abort_flag) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * kTileCols;
                    for (int k = 0; k < g.k_iters; ++k) {
                        if (!ready && !ptx::mbar_wait(&full[stage], phase, g.wait_budget)) { ok = false; break; }
                        ptx::tc_fence_after();
                        const int next_stage = stage + 1 == kStages ? 0 : stage + 1;
                        const uint32_t next_phase = stage + 1 == kStages ? phase ^ 1 : phase;
                        ready = ptx::mbar_test_wait(&full[next_stage], next_phase);
                        const uint32_t sA = ptx::smem_u32(smem + stage * kStageBytes);
                        const uint64_t da = A_MN ? ptx::smem_desc_mn_sw128(sA, kMnBoxBytes) : ptx::smem_desc_k_sw128(sA);
                        const uint64_t db = B_MN ? ptx::smem_desc_mn_sw128(sA + kABytes, kMnBoxBytes)
                                                 : ptx::smem_desc_k_sw128(sA + kABytes);
                        // start-address step (16-byte units) per 16 values of K: 32 B inside a K-major swizzle row,
                        // 16 rows x 128 B for an MN-major operand
                        constexpr uint32_t step_a = A_MN ? (16 * 128) >> 4 : 2;
                        constexpr uint32_t step_b = B_MN ? (16 * 128) >> 4 : 2;
                        // the shared-memory descriptor counts addresses in 16-byte units
#pragma unroll
                        for (int nb = 0; nb < NB; ++nb) {
#pragma unroll
                            for (int kk = 0; kk < kTileK / 16; ++kk)
                                ptx::mma_bf16_ss_on<CTAS>(d_tmem + nb * kTileN, da + step_a * kk,
                                                          db + static_cast<uint64_t>(nb * (kBBytes >> 4)) + step_b * kk, idesc,
                                                          (k | kk) != 0 ? 1u : 0u);
                        }
                        ptx::tc_commit_on<CTAS>(&empty[stage]);
                        stage = next_stage;
                        phase = next_phase;
                    }
                    if (!ok) break;
                    ptx::tc_commit_on<CTAS>(&acc_full[acc]);
                    if (++acc == kAccStages) { acc = 0; acc_phase ^= 1; }
                }
            }
            if (!ok) { *abort_flag = 1; atomicOr(g.status, kStatusTimeout); }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: thread = one row (both CTAs)
        const int quarter = warp & 3;                      // TMEM lanes this warp may touch: 32*quarter ..
        const int row_in_tile = static_cast<int>(cta_rank) * kCtaM + quarter * 32 + lane;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        const uint64_t pol_st = ptx::l2_policy((g.l2_hints >> 4) & 3);
        for (int it = 0; ok; ++it) {
            Unit t;
            bool valid;
            if (!next_unit<EPI>(g, it, pair, n_pairs, gm, t, valid)) break;
            if (!valid) continue;
            const int row = t.m_tile * C::kTileRows + row_in_tile;        // relative to a_row0
            const bool row_ok = row < g.m_rows;

            // per-row state
            float run_m = kNegBig, z_tgt = kNegBig;
            uint64_t run_s2 = 0ull, run_t2 = 0ull;           // (even, odd) partial sums of e and e*v
            int tgt = -1;
            float ca = 0.f, cb = 0.f, lse = 0.f, ent = 0.f;
            if (EPI == kEpiSoftmaxStats || EPI == kEpiLogitGrad) {
                if (row_ok) tgt = g.target_p[g.a_row0 + row] - g.vocab0;     // column index relative to b_row0
            }
            if (EPI == kEpiLogitGrad && row_ok) {
                ca = g.coef_a[g.a_row0 + row];
                cb = g.coef_b[g.a_row0 + row];
                lse = g.row_lse[g.a_row0 + row];
                ent = g.row_ent[g.a_row0 + row];
            }
            const float c2 = g.scale * kLog2e;
            // per-row constants of the logit-gradient epilogue (see there)
            float gshift = 0.f, gA = 0.f, gB = 0.f;
            unsigned gsign = 0u;
            if (EPI == kEpiLogitGrad) {
                gshift = -lse * kLog2e;
                if (!g.has_ent) {
                    gshift += __log2f(fabsf(ca));              // -inf for a == 0: every exp2 below gives 0
                    gsign = ca > 0.f ? 0x80008000u : 0u;
                } else {
                    gA = -fmaf(cb, ent - lse, ca);
                    gB = -cb * g.scale;
                }
            }

            for (int ni = t.n_begin; ni < t.n_end && ok; ++ni) {
                const int nt = t.rev ? t.n_begin + t.n_end - 1 - ni : ni;
                if (!ptx::mbar_wait(&acc_full[acc], acc_phase, g.wait_budget) || *abort_flag) { ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * kTileCols;
                const int mma_n = EPI == kEpiAccumF32 ? g.mma_n : kTileN;     // columns per MMA block (<= 256)
                const int col0 = nt * (NB * mma_n);
                const int per_block = mma_n / 32;
#pragma unroll 1
                for (int c = 0; c < NB * per_block; ++c) {
                    const int cbase = col0 + c * 32;            // block nb of a two-block tile starts at col0 + nb * mma_n
                    if (cbase >= g.n_cols) break;               // uniform across the CTA
                    uint32_t rr[32];
                    // ... and sits at tensor-memory column nb * 256 whatever mma_n is
                    ptx::tmem_ld_32x32(taddr + (NB == 1 ? c * 32 : (c / per_block) * kTileN + (c % per_block) * 32), rr);
                    ptx::tmem_ld_wait();
                    float v[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(rr[j]);
                    const int n_here = min(32, g.n_cols - cbase);

                    if (EPI == kEpiSoftmaxStats) {
                        if (n_here < 32) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) if (j >= n_here) v[j] = kNegBig;
                        }
                        float cm = ptx::max3(v[0], v[1], v[2]);
#pragma unroll
                        for (int j = 3; j < 31; j += 2) cm = ptx::max3(cm, v[j], v[j + 1]);
                        cm = fmaxf(cm, v[31]);
                        const float new_m = fmaxf(run_m, cm);
                        const float resc = ptx::ex2((run_m - new_m) * c2);
                        const uint64_t resc2 = ptx::pack2(resc, resc);
                        run_s2 = ptx::mul2(run_s2, resc2);
                        run_t2 = ptx::mul2(run_t2, resc2);
                        run_m = new_m;
                        const float shift = -new_m * c2;
                        const uint64_t shift2 = ptx::pack2(shift, shift), c22 = ptx::pack2(c2, c2);
                        // two logits per instruction: e = 2^(v*c2 + shift); sum e; sum e*v (even / odd partial sums)
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            const uint64_t x = ptx::pack2(v[j], v[j + 1]);
                            float a0, a1;
                            ptx::unpack2(ptx::fma2(x, c22, shift2), a0, a1);
                            const uint64_t e = ptx::pack2(ptx::ex2(a0), ptx::ex2(a1));
                            run_s2 = ptx::add2(run_s2, e);
                            run_t2 = ptx::fma2(e, x, run_t2);
                        }
                        const int jt = tgt - cbase;
                        if (jt >= 0 && jt < 32) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) if (j == jt) z_tgt = v[j];
                        }
                        if (g.Z != nullptr && row_ok) {
                            // keep the scaled logits of this bounded block of rows (bf16), grouped by vocabulary
                            // chunk, for a backward pass that does not recompute them
                            int zc = cbase / g.z_chunk_cols;
                            zc = zc < g.z_chunks - 1 ? zc : g.z_chunks - 1;
                            __nv_bfloat16* dst = g.Z + zc * g.z_chunk_stride + static_cast<long long>(row) * g.ldz +
                                                 (cbase - zc * g.z_chunk_cols);
                            unsigned zp[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) zp[j] = pack_bf16(v[2 * j] * g.scale, v[2 * j + 1] * g.scale);
                            if (n_here == 32 && g.g_wide_store) {
                                ptx::st_global_v8(dst, zp[0], zp[1], zp[2], zp[3], zp[4], zp[5], zp[6], zp[7]);
                                ptx::st_global_v8(dst + 16, zp[8], zp[9], zp[10], zp[11], zp[12], zp[13], zp[14], zp[15]);
                            } else {
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    if (q * 8 < n_here)
                                        *reinterpret_cast<uint4*>(dst + q * 8) =
                                            make_uint4(zp[4 * q], zp[4 * q + 1], zp[4 * q + 2], zp[4 * q + 3]);
                                }
                            }
                        }
                    } else if (EPI == kEpiLogitGrad) {
                        // G = -p*(a + b*(z - lse + H)) (+ a at the target), z = scale*acc, p = exp(z - lse), written
                        // with as few instructions per logit as possible (the epilogue shares issue slots and power
                        // with the MMAs of the next tile):
                        //   b == 0 for the whole launch:  |G| = exp2(acc*c2 + (shift + log2|a|)), sign(G) = -sign(a)
                        //                                 -> one FMA and one exp2 per logit, sign set on the packed pair
                        //   otherwise:                    G = p * (A + B*acc), A = -(a + b*(H - lse)), B = -b*scale
                        unsigned packed[16];
                        const uint64_t c22 = ptx::pack2(c2, c2), gshift2 = ptx::pack2(gshift, gshift);
                        if (!g.has_ent) {
#pragma unroll
                            for (int j = 0; j < 32; j += 2) {
                                float a0, a1;
                                ptx::unpack2(ptx::fma2(ptx::pack2(v[j], v[j + 1]), c22, gshift2), a0, a1);
                                packed[j >> 1] = pack_bf16(ptx::ex2(a0), ptx::ex2(a1)) ^ gsign;
                            }
                        } else {
                            const uint64_t gA2 = ptx::pack2(gA, gA), gB2 = ptx::pack2(gB, gB);
#pragma unroll
                            for (int j = 0; j < 32; j += 2) {
                                const uint64_t x = ptx::pack2(v[j], v[j + 1]);
                                float a0, a1, o0, o1;
                                ptx::unpack2(ptx::fma2(x, c22, gshift2), a0, a1);
                                ptx::unpack2(ptx::mul2(ptx::pack2(ptx::ex2(a0), ptx::ex2(a1)), ptx::fma2(gB2, x, gA2)), o0, o1);
                                packed[j >> 1] = pack_bf16(o0, o1);
                            }
                        }
                        const int jt = tgt - cbase;
                        if (jt >= 0 && jt < 32) {                 // the target logit of this row: add a (rare branch)
                            float vt = 0.f;
#pragma unroll
                            for (int j = 0; j < 32; ++j) if (j == jt) vt = v[j];
                            const float z = vt * g.scale;
                            const float pt = ptx::ex2(fmaf(z, kLog2e, -lse * kLog2e));
                            const float gt = fmaf(-pt, fmaf(cb, z + (ent - lse), ca), ca);
                            const unsigned bits = static_cast<unsigned>(__bfloat16_as_ushort(__float2bfloat16_rn(gt)));
                            const unsigned keep = (jt & 1) ? 0x0000ffffu : 0xffff0000u;
                            const unsigned put = (jt & 1) ? (bits << 16) : bits;
                            const int jp = jt >> 1;
#pragma unroll
                            for (int j = 0; j < 16; ++j) packed[j] = (j == jp) ? ((packed[j] & keep) | put) : packed[j];
                        }
                        if (row_ok) {
                            __nv_bfloat16* dst = g.G + static_cast<long long>(row) * g.ldg + cbase;
                            if (n_here == 32 && g.g_wide_store) {
                                // two full 32-byte sectors per thread instead of four half sectors
                                ptx::st_global_v8_hint(dst, packed[0], packed[1], packed[2], packed[3], packed[4], packed[5],
                                                       packed[6], packed[7], pol_st);
                                ptx::st_global_v8_hint(dst + 16, packed[8], packed[9], packed[10], packed[11], packed[12],
                                                       packed[13], packed[14], packed[15], pol_st);
                            } else {
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    if (q * 8 < n_here)
                                        *reinterpret_cast<uint4*>(dst + q * 8) =
                                            make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
                                }
                            }
                        }
                    } else {
                        if (row_ok) {
                            float* dst = g.C + static_cast<long long>(row) * g.ldc + cbase;
#pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                if (q * 4 < n_here) {
                                    float4 o = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                                    if (NB == 2 && g.beta) {
                                        // one owner per element per launch and launches are stream-ordered, so the
                                        // sum is the same single rounded addition as load-add-store
                                        ptx::red_add_v4_f32(dst + q * 4, o);
                                        continue;
                                    }
                                    if (g.beta) {
                                        const float4 old = *reinterpret_cast<const float4*>(dst + q * 4);
                                        o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                                    }
                                    *reinterpret_cast<float4*>(dst + q * 4) = o;
                                }
                            }
                        }
                    }
                }
                // release the accumulator stage to the MMA issuer in the even CTA
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (CTAS == 2) ptx::mbar_arrive_cluster(ptx::mapa(ptx::smem_u32(&acc_empty[acc]), 0));
                    else ptx::mbar_arrive(&acc_empty[acc]);
                }
                if (++acc == kAccStages) { acc = 0; acc_phase ^= 1; }
            }
            if (EPI == kEpiSoftmaxStats && ok && row_ok) {
                float s0, s1, t0, t1;
                ptx::unpack2(run_s2, s0, s1);
                ptx::unpack2(run_t2, t0, t1);
                const long long at = t.m_tile >= g.last_m0
                                         ? g.last_stats_off + t.split * g.last_pitch + (row - g.last_m0 * C::kTileRows)
                                         : t.split * g.stats_pitch + row;
                g.stats[at] = make_float4(run_m, s0 + s1, t0 + t1, z_tgt);
            }
        }
        if (!ok) { *abort_flag = 1; atomicOr(g.status, kStatusTimeout); }
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    if (*abort_flag) {
        // copies issued before the abort may still be landing in shared memory: give them time
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000) { }
    }
    ptx::tc_fence_before();
    if (CTAS == 2) ptx::cluster_sync_all();   // neither CTA leaves (or frees tensor memory) while its peer may touch it
    else __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        if (CTAS == 2) ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
        else ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}


template <int EPI, bool A_MN, bool B_MN, int CTAS, int NB = 1>
cudaError_t set_attr() {
    return cudaFuncSetAttribute(k_gemm<EPI, A_MN, B_MN, CTAS, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                Cfg<CTAS, NB>::kSmemBytes);
}

template <int EPI, bool A_MN, bool B_MN, int CTAS, int NB = 1>
cudaError_t launch(const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmArgs& args, int workers, cudaStream_t stream) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(workers * CTAS, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = Cfg<CTAS, NB>::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CTAS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_gemm<EPI, A_MN, B_MN, CTAS, NB>, tmA, tmB, args);
}

}  // namespace

cudaError_t gemm_set_attributes() {
    cudaError_t e;
    if ((e = set_attr<kEpiSoftmaxStats, false, false, 1>()) != cudaSuccess) return e;
    if ((e = set_attr<kEpiSoftmaxStats, false, false, 2>()) != cudaSuccess) return e;
    if ((e = set_attr<kEpiLogitGrad, false, false, 1>()) != cudaSuccess) return e;
    if ((e = set_attr<kEpiLogitGrad, false, false, 2>()) != cudaSuccess) return e;
    if ((e = set_attr<kEpiAccumF32, false, true, 1>()) != cudaSuccess) return e;
    if ((e = set_attr<kEpiAccumF32, false, true, 2>()) != cudaSuccess) return e;
    if ((e = set_attr<kEpiAccumF32, true, true, 1>()) != cudaSuccess) return e;
    if ((e = set_attr<kEpiAccumF32, true, true, 2>()) != cudaSuccess) return e;
    if ((e = set_attr<kEpiAccumF32, false, true, 2, 2>()) != cudaSuccess) return e;
    return set_attr<kEpiAccumF32, true, true, 2, 2>();
}

int gemm_tile_rows(int ctas) { return kCtaM * ctas; }
int gemm_mma_n(int n_cols) {
    const int blocks = (n_cols + kTileN - 1) / kTileN;
    const int per = (n_cols + blocks - 1) / blocks;
    return (per + 31) / 32 * 32;
}

cudaError_t launch_gemm(GemmEpilogue epi, bool a_mn, int ctas, const CUtensorMap& tmA, const CUtensorMap& tmB,
                        const GemmArgs& args, int sm_count, cudaStream_t stream, bool wide, int workers_known) {
    // softmax: one round handles group_m row tiles x n_splits; other epilogues: plain striding over all tiles.  With the
    // row extent known on the device only, the launch takes the whole machine; workers without a unit leave at once.
    const int max_workers = sm_count / ctas;                                   // one CTA per SM
    int workers = workers_known > 0 && workers_known < max_workers ? workers_known : max_workers;
    if (args.span.plan == nullptr) {
        const long long units = epi == kEpiSoftmaxStats
                                    ? static_cast<long long>(args.group_m < args.m_tiles ? args.group_m : args.m_tiles) * args.n_splits
                                    : static_cast<long long>(args.m_tiles) * args.n_tiles;
        if (units <= 0 || args.m_tiles <= 0 || args.k_iters <= 0) return cudaSuccess;
        workers = static_cast<int>(units < max_workers ? units : max_workers);
    }
    if (epi == kEpiAccumF32 && (args.mma_n < 32 || args.mma_n > kTileN || args.mma_n % 32 != 0)) return cudaErrorInvalidValue;
    const bool two = ctas == 2;
    switch (epi) {
        case kEpiSoftmaxStats:
            return two ? launch<kEpiSoftmaxStats, false, false, 2>(tmA, tmB, args, workers, stream)
                       : launch<kEpiSoftmaxStats, false, false, 1>(tmA, tmB, args, workers, stream);
        case kEpiLogitGrad:
            return two ? launch<kEpiLogitGrad, false, false, 2>(tmA, tmB, args, workers, stream)
                       : launch<kEpiLogitGrad, false, false, 1>(tmA, tmB, args, workers, stream);
        default:   // fp32 accumulate: B is always MN-major (W or hidden read in place), A is G either way round
            if (wide && two)
                return a_mn ? launch<kEpiAccumF32, true, true, 2, 2>(tmA, tmB, args, workers, stream)
                            : launch<kEpiAccumF32, false, true, 2, 2>(tmA, tmB, args, workers, stream);
            if (a_mn)
                return two ? launch<kEpiAccumF32, true, true, 2>(tmA, tmB, args, workers, stream)
                           : launch<kEpiAccumF32, true, true, 1>(tmA, tmB, args, workers, stream);
            return two ? launch<kEpiAccumF32, false, true, 2>(tmA, tmB, args, workers, stream)
                       : launch<kEpiAccumF32, false, true, 1>(tmA, tmB, args, workers, stream);
    }
}

}  // namespace unity
