// Persistent, warp-specialised bf16 GEMM for sm_100a:  C[m, n] = sum_k A[m, k] * B[n, k], each operand
// either K-major ([rows, K] in memory) or MN-major ([K, rows] in memory), so no operand is ever transposed in HBM.
//
//   warp 0      : TMA producer  - streams 128x64 (A) and 256x64 (B) bf16 slabs into a 4-stage shared-memory ring
//   warp 1      : MMA issuer    - one thread issues tcgen05.mma (128x256x16) into one of two 256-column TMEM
//                                 accumulator stages and commits completion to mbarriers
//   warps 2..5  : epilogue      - each thread owns one accumulator row (one TMEM lane), drains it 32 columns at
//                                 a time with tcgen05.ld while the MMA warp already fills the other stage
//
// Three epilogues share the main loop:
//   softmax statistics : running (max, sum exp, sum exp*z, target logit) per row across a sweep of vocabulary
//                        tiles; nothing of size rows x vocabulary is ever written
//   logit gradient     : dL/dz = a*(onehot - p) - b*p*(z - lse + H) in bf16 for a bounded chunk
//   fp32 accumulate    : C (+)= acc
// Every mbarrier wait is bounded; on expiry the CTA records a timeout status, all roles leave their loops and
// the kernel frees its tensor memory and returns.
#include "internal.h"
#include "ptx.cuh"

namespace unity {

namespace {

constexpr int kStages = 4;
constexpr int kABytes = kTileM * kTileK * 2;              // 16 KiB
constexpr int kBBytes = kTileN * kTileK * 2;              // 32 KiB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kAccStages = 2;
constexpr int kTmemCols = kAccStages * kTileN;            // 512: all of tensor memory
constexpr int kBarBytes = 256;
constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kBarBytes;
constexpr int kThreads = 192;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegBig = -3.0e38f;

struct Unit {
    int m_tile, n_begin, n_end, split;
};

// Work decomposition.  Softmax: a unit is (row tile, vocabulary split); groups of `gm` row tiles x all splits
// are laid out consecutively so that one wave of CTAs shares a small set of A tiles (L2 resident) while the
// splits stream disjoint parts of B.  Other epilogues: one output tile per unit, m fastest inside groups of
// `gm` row tiles.
template <int EPI>
__device__ __forceinline__ int num_units(const GemmArgs& g) {
    return EPI == kEpiSoftmaxStats ? g.m_tiles * g.n_splits : g.m_tiles * g.n_tiles;
}
template <int EPI>
__device__ __forceinline__ Unit get_unit(const GemmArgs& g, int u, int gm) {
    Unit t;
    if (EPI == kEpiSoftmaxStats) {
        const int per_group = gm * g.n_splits;
        const int grp = u / per_group, r = u - grp * per_group;
        const int m0 = grp * gm;
        const int gm_here = min(gm, g.m_tiles - m0);
        t.split = r / gm_here;
        t.m_tile = m0 + (r - t.split * gm_here);
        t.n_begin = t.split * g.tiles_per_split;
        t.n_end = min(t.n_begin + g.tiles_per_split, g.n_tiles);
    } else {
        const int per_group = gm * g.n_tiles;
        const int grp = u / per_group, r = u - grp * per_group;
        const int m0 = grp * gm;
        const int gm_here = min(gm, g.m_tiles - m0);
        const int nt = r / gm_here;
        t.m_tile = m0 + (r - nt * gm_here);
        t.n_begin = nt;
        t.n_end = nt + 1;
        t.split = 0;
    }
    return t;
}

__device__ __forceinline__ unsigned pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<unsigned*>(&v);
}

// Operand layouts.  K-major: the operand is stored [rows, K] and a stage holds one box of (rows x 64 K).
// MN-major: the operand is stored [K, rows] (rows contiguous) and a stage holds rows/64 boxes of (64 rows x 64 K),
// 8 KiB each, one after the other; the matrix descriptor then has leading byte offset 8 KiB (next 64 rows) and
// stride byte offset 1 KiB (next 8 values of K), and 16 values of K further is 2 KiB further.
constexpr int kMnBoxBytes = 64 * kTileK * 2;

template <int EPI, bool A_MN, bool B_MN>
__global__ void __launch_bounds__(kThreads, 1)
k_gemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
    uint64_t* full = bars;                       // [kStages]  TMA bytes landed
    uint64_t* empty = bars + kStages;            // [kStages]  MMAs that read the stage have completed
    uint64_t* acc_full = bars + 2 * kStages;     // [2]        accumulator stage complete
    uint64_t* acc_empty = acc_full + kAccStages; // [2]        accumulator stage drained by the epilogue
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + kAccStages);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
        for (int s = 0; s < kAccStages; ++s) { ptx::mbar_init(&acc_full[s], 1); ptx::mbar_init(&acc_empty[s], 4); }
        *abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmB);
    }
    if (warp == 1) {
        ptx::tmem_alloc(tmem_slot, kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int n_units = num_units<EPI>(g);
    const int gm = max(1, g.group_m);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
                const Unit t = get_unit<EPI>(g, u, gm);
                const int a_row = g.a_row0 + t.m_tile * kTileM;
                for (int nt = t.n_begin; nt < t.n_end && ok; ++nt) {
                    const int b_row = g.b_row0 + nt * kTileN;
                    for (int k = 0; k < g.k_iters; ++k) {
                        if (!ptx::mbar_wait(&empty[stage], phase ^ 1, kWaitBudgetCycles) || *abort_flag) { ok = false; break; }
                        uint8_t* sA = smem + stage * kStageBytes;
                        ptx::mbar_arrive_expect_tx(&full[stage], kStageBytes);
                        if (A_MN) {
#pragma unroll
                            for (int j = 0; j < kTileM / 64; ++j)
                                ptx::tma_load_2d(sA + j * kMnBoxBytes, &tmA, &full[stage], a_row + j * 64, g.a_k0 + k * kTileK);
                        } else {
                            ptx::tma_load_2d(sA, &tmA, &full[stage], g.a_k0 + k * kTileK, a_row);
                        }
                        if (B_MN) {
#pragma unroll
                            for (int j = 0; j < kTileN / 64; ++j)
                                ptx::tma_load_2d(sA + kABytes + j * kMnBoxBytes, &tmB, &full[stage], b_row + j * 64,
                                                 g.b_k0 + k * kTileK);
                        } else {
                            ptx::tma_load_2d(sA + kABytes, &tmB, &full[stage], g.b_k0 + k * kTileK, b_row);
                        }
                        if (++stage == kStages) { stage = 0; phase ^= 1; }
                    }
                }
            }
            if (!ok) { *abort_flag = 1; atomicOr(g.status, kStatusTimeout); }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_bf16_f32(kTileM, kTileN) | (A_MN ? (1u << 15) : 0u) | (B_MN ? (1u << 16) : 0u);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
                const Unit t = get_unit<EPI>(g, u, gm);
                for (int nt = t.n_begin; nt < t.n_end && ok; ++nt) {
                    if (!ptx::mbar_wait(&acc_empty[acc], acc_phase ^ 1, kWaitBudgetCycles) || *abort_flag) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * kTileN;
                    for (int k = 0; k < g.k_iters; ++k) {
                        if (!ptx::mbar_wait(&full[stage], phase, kWaitBudgetCycles) || *abort_flag) { ok = false; break; }
                        ptx::tc_fence_after();
                        const uint32_t sA = ptx::smem_u32(smem + stage * kStageBytes);
                        const uint64_t da = A_MN ? ptx::smem_desc_mn_sw128(sA, kMnBoxBytes) : ptx::smem_desc_k_sw128(sA);
                        const uint64_t db = B_MN ? ptx::smem_desc_mn_sw128(sA + kABytes, kMnBoxBytes)
                                                 : ptx::smem_desc_k_sw128(sA + kABytes);
                        // start-address step (16-byte units) per 16 values of K: 32 B inside a K-major swizzle row,
                        // 16 rows x 128 B for an MN-major operand
                        constexpr uint32_t step_a = A_MN ? (16 * 128) >> 4 : 2;
                        constexpr uint32_t step_b = B_MN ? (16 * 128) >> 4 : 2;
#pragma unroll
                        for (int kk = 0; kk < kTileK / 16; ++kk)
                            ptx::mma_bf16_ss(d_tmem, da + step_a * kk, db + step_b * kk, idesc, (k | kk) != 0 ? 1u : 0u);
                        ptx::tc_commit(&empty[stage]);
                        if (++stage == kStages) { stage = 0; phase ^= 1; }
                    }
                    if (!ok) break;
                    ptx::tc_commit(&acc_full[acc]);
                    if (++acc == kAccStages) { acc = 0; acc_phase ^= 1; }
                }
            }
            if (!ok) { *abort_flag = 1; atomicOr(g.status, kStatusTimeout); }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: thread = one row
        const int quarter = warp & 3;                      // TMEM lanes this warp may touch: 32*quarter ..
        const int row_in_tile = quarter * 32 + lane;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
            const Unit t = get_unit<EPI>(g, u, gm);
            const int row = t.m_tile * kTileM + row_in_tile;        // relative to a_row0
            const bool row_ok = row < g.m_rows;

            // per-row state
            float run_m = kNegBig, run_s = 0.f, run_t = 0.f, z_tgt = kNegBig;
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

            for (int nt = t.n_begin; nt < t.n_end && ok; ++nt) {
                if (!ptx::mbar_wait(&acc_full[acc], acc_phase, kWaitBudgetCycles) || *abort_flag) { ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * kTileN;
                const int col0 = nt * kTileN;
#pragma unroll 1
                for (int c = 0; c < kTileN / 32; ++c) {
                    const int cbase = col0 + c * 32;
                    if (cbase >= g.n_cols) break;               // uniform across the CTA
                    uint32_t rr[32];
                    ptx::tmem_ld_32x32(taddr + c * 32, rr);
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
                        float cm = v[0];
#pragma unroll
                        for (int j = 1; j < 32; ++j) cm = fmaxf(cm, v[j]);
                        const float new_m = fmaxf(run_m, cm);
                        const float resc = exp2f((run_m - new_m) * c2);
                        run_s *= resc;
                        run_t *= resc;
                        run_m = new_m;
                        const float shift = -new_m * c2;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float e = exp2f(fmaf(v[j], c2, shift));
                            run_s += e;
                            run_t = fmaf(e, v[j], run_t);
                        }
                        const int jt = tgt - cbase;
                        if (jt >= 0 && jt < 32) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) if (j == jt) z_tgt = v[j];
                        }
                    } else if (EPI == kEpiLogitGrad) {
                        // G = -p*(a + b*(z - lse + H)) (+ a at the target), z = scale*acc, p = exp(z - lse)
                        const float shift = -lse * kLog2e;
                        const float hl = ent - lse;
                        unsigned packed[16];
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            float o[2];
#pragma unroll
                            for (int q = 0; q < 2; ++q) {
                                const float z = v[j + q] * g.scale;
                                const float p = exp2f(fmaf(z, kLog2e, shift));
                                float gg = -p * fmaf(cb, z + hl, ca);
                                if (cbase + j + q == tgt) gg += ca;
                                o[q] = gg;
                            }
                            packed[j >> 1] = pack_bf16(o[0], o[1]);
                        }
                        if (row_ok) {
                            __nv_bfloat16* dst = g.G + static_cast<long long>(row) * g.ldg + cbase;
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                if (q * 8 < n_here)
                                    *reinterpret_cast<uint4*>(dst + q * 8) =
                                        make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
                            }
                        }
                    } else {
                        if (row_ok) {
                            float* dst = g.C + static_cast<long long>(row) * g.ldc + cbase;
#pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                if (q * 4 < n_here) {
                                    float4 o = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
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
                // release the accumulator stage to the MMA warp
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&acc_empty[acc]);
                if (++acc == kAccStages) { acc = 0; acc_phase ^= 1; }
            }
            if (EPI == kEpiSoftmaxStats && ok && row_ok)
                g.stats[t.split * g.stats_pitch + row] = make_float4(run_m, run_s, run_t, z_tgt);
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
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

cudaError_t gemm_set_attributes() {
    cudaError_t e;
    e = cudaFuncSetAttribute(k_gemm<kEpiSoftmaxStats, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_gemm<kEpiLogitGrad, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_gemm<kEpiAccumF32, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(k_gemm<kEpiAccumF32, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}

cudaError_t launch_gemm(GemmEpilogue epi, bool a_mn, const CUtensorMap& tmA, const CUtensorMap& tmB,
                        const GemmArgs& args, int sm_count, cudaStream_t stream) {
    const long long units = epi == kEpiSoftmaxStats ? static_cast<long long>(args.m_tiles) * args.n_splits
                                                    : static_cast<long long>(args.m_tiles) * args.n_tiles;
    if (units <= 0 || args.k_iters <= 0) return cudaSuccess;
    const int grid = static_cast<int>(units < sm_count ? units : sm_count);
    switch (epi) {
        case kEpiSoftmaxStats:
            k_gemm<kEpiSoftmaxStats, false, false><<<grid, kThreads, kSmemBytes, stream>>>(tmA, tmB, args);
            break;
        case kEpiLogitGrad:
            k_gemm<kEpiLogitGrad, false, false><<<grid, kThreads, kSmemBytes, stream>>>(tmA, tmB, args);
            break;
        default:   // fp32 accumulate: B is always MN-major (W or hidden read in place), A is G either way round
            if (a_mn) k_gemm<kEpiAccumF32, true, true><<<grid, kThreads, kSmemBytes, stream>>>(tmA, tmB, args);
            else k_gemm<kEpiAccumF32, false, true><<<grid, kThreads, kSmemBytes, stream>>>(tmA, tmB, args);
            break;
    }
    return cudaGetLastError();
}

}  // namespace unity
