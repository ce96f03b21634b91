// Streaming (HBM / latency bound) kernels of libunity: role-level advantage, routing of response
// tokens to their model through the agent-to-model table, row packing, per-token PPO
// terms with fixed-order reductions, and the dHidden write-back.  No floating-point atomics anywhere:
// every reduction has a fixed order, so results are bitwise reproducible.
#include "internal.h"

namespace unity {

namespace {

constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
__device__ __forceinline__ int warp_sum_int(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}

// Invocation that owns token `tok`: the s with cu[s] <= tok < cu[s+1] (zero-length invocations are skipped).
__device__ __forceinline__ int find_invocation(const int64_t* __restrict__ cu, int n_inv, long long tok) {
    int lo = 0, hi = n_inv;   // number of entries cu[1..n_inv] that are <= tok
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (cu[mid + 1] <= tok) lo = mid + 1; else hi = mid;
    }
    return min(lo, n_inv - 1);
}

// ------------------------------------------------------------------------------------------------
// Stage 1: advantage
// ------------------------------------------------------------------------------------------------
// Segment statistics without any ordering assumption.  Invocations of a (group, role) segment may sit anywhere in the
// batch (buffers fill in arrival order), so nothing here sweeps index ranges: every pass is one thread per invocation
// plus integer atomics on a per-segment table.  Integer addition is associative, so the result does not depend on the
// order in which the atomics land: the statistics are exact on the segment's grid and bitwise reproducible.
//   pass 1 : r_s, segment id; per segment the member count n and max |r|
//   pass 2 : q_s = r_s on the segment's integer grid; per segment S = sum q (64 bits) and Q = sum q^2 (128 bits)
//   pass 3 : n Q - S^2 = n * sum (q - S/n)^2 exactly, in 128-bit integers (no rounding, hence none of the cancellation
//            that makes E[r^2] - mean^2 unusable in floating point; 0 for a segment whose rewards are all equal);
//            mean, sigma and the advantages (n q_s - S) / (n (sigma + eps)) follow in fp64 and are rounded to fp32
// Grid of a segment with n <= 2^L members and max |r| < 2^(E+1): multiples of 2^-shift, shift = B - (E + 1), with
// B = min(61 - L, (125 - 3 L) / 2) bits per value, so that S stays below 2^62 and n Q below 2^127.  For segments of
// up to 64 members that is 53 or more bits (every fp32 reward within 2^29 of the largest is exact).
// The three passes run as ONE cooperative launch with a bounded grid barrier between them (all blocks are resident by
// construction of the launch); a device without cooperative launch gets three launches of the same code.
struct SegTable {
    int* cnt;
    unsigned* maxbits;
    long long* sum;
    unsigned long long *sqlo, *sqhi;
};
constexpr size_t kSegHeaderBytes = 256;     // the table starts with the barrier counter of the fused launch
__device__ __forceinline__ SegTable seg_table(const AdvArgs& a) {
    const size_t n = static_cast<size_t>(a.n_groups) * a.n_roles;
    SegTable t;
    t.cnt = reinterpret_cast<int*>(static_cast<char*>(a.seg_table) + kSegHeaderBytes);
    t.maxbits = reinterpret_cast<unsigned*>(t.cnt + n);
    t.sum = reinterpret_cast<long long*>(t.maxbits + n);
    t.sqlo = reinterpret_cast<unsigned long long*>(t.sum + n);
    t.sqhi = t.sqlo + n;
    return t;
}
__device__ __forceinline__ int seg_shift(unsigned maxbits, int cnt) {
    const int E = ilogbf(__uint_as_float(maxbits));              // max |r| > 0 (subnormals included)
    const int L = cnt > 1 ? 32 - __clz(cnt - 1) : 0;             // cnt <= 2^L
    const int B = min(61 - L, (125 - 3 * L) / 2);
    return B - (E + 1);
}
__device__ __forceinline__ long long seg_quantise(float r, int shift) {
    return __double2ll_rn(ldexp(static_cast<double>(r), shift));
}

__device__ __forceinline__ void adv_pass_combine(const AdvArgs& a, int s) {
    const int v = a.inv_role[s], g = a.inv_group[s];
    bool ok = (v >= 0 && v < a.n_roles && g >= 0 && g < a.n_groups);
    float rj = 0.f;
    if (a.r_traj != nullptr) {
        const int t = a.inv_traj[s];
        if (t >= 0 && t < a.n_traj) rj = a.r_traj[t]; else ok = false;
    }
    float r = 0.f;
    int seg = -1;
    if (ok) {
        const float ln = a.has_lam ? a.lam[v * 3 + 0] : 1.f;
        const float lt = a.has_lam ? a.lam[v * 3 + 1] : 1.f;
        const float lj = a.has_lam ? a.lam[v * 3 + 2] : 1.f;
        const float rn = a.r_node ? a.r_node[s] : 0.f;
        const float rt = a.r_turn ? a.r_turn[s] : 0.f;
        r = __fadd_rn(__fadd_rn(__fmul_rn(ln, rn), __fmul_rn(lt, rt)), __fmul_rn(lj, rj));
        seg = g * a.n_roles + v;
        const SegTable t = seg_table(a);
        atomicAdd(&t.cnt[seg], 1);
        atomicMax(&t.maxbits[seg], __float_as_uint(fabsf(r)));   // bit patterns of non-negative floats order like the floats
    } else {
        atomicOr(a.status, kStatusBadIndex);
    }
    a.r_scratch[s] = r;
    a.seg_scratch[s] = seg;
}

__device__ __forceinline__ void adv_pass_sums(const AdvArgs& a, int s) {
    const int seg = a.seg_scratch[s];
    if (seg < 0) return;
    const SegTable t = seg_table(a);
    // (the table is written by atomics of other blocks in the pass before: read it from L2, not through L1)
    const unsigned mb = __ldcg(&t.maxbits[seg]);
    if (mb == 0u) return;                                        // every reward of the segment is zero
    const long long q = seg_quantise(a.r_scratch[s], seg_shift(mb, __ldcg(&t.cnt[seg])));
    if (q == 0) return;
    atomicAdd(reinterpret_cast<unsigned long long*>(&t.sum[seg]), static_cast<unsigned long long>(q));
    const unsigned long long m = static_cast<unsigned long long>(q < 0 ? -q : q);
    const unsigned long long lo = m * m, hi = __umul64hi(m, m);
    // 128-bit accumulation with two 64-bit atomics: the low word's wrap-arounds are carried into the high word by
    // whoever caused them, so the final pair is the exact sum whatever the order
    const unsigned long long old = atomicAdd(&t.sqlo[seg], lo);
    const unsigned long long carry = (old + lo < old) ? 1ull : 0ull;
    if (hi + carry != 0ull) atomicAdd(&t.sqhi[seg], hi + carry);
}

// Index i finishes invocation i (advantage) and segment i (mean and sigma for the caller).
__device__ __forceinline__ void adv_pass_finish(const AdvArgs& a, int i) {
    const int n_seg = a.n_groups * a.n_roles;
    const SegTable t = seg_table(a);
    auto stats = [&](int seg, double& mean, double& sigma, double& unit, int& cnt, int& shift) {
        cnt = __ldcg(&t.cnt[seg]);
        const unsigned mb = __ldcg(&t.maxbits[seg]);
        mean = 0.0; sigma = 0.0; unit = 0.0; shift = 0;
        if (cnt == 0 || mb == 0u) return;
        shift = seg_shift(mb, cnt);
        unit = ldexp(1.0 / static_cast<double>(cnt), -shift);            // value of one step of n q - S
        const long long S = __ldcg(&t.sum[seg]);
        mean = static_cast<double>(S) * unit;
        const int dof = cnt - a.ddof;
        if (dof > 0) {
            const unsigned __int128 Q = (static_cast<unsigned __int128>(__ldcg(&t.sqhi[seg])) << 64) | __ldcg(&t.sqlo[seg]);
            const unsigned long long absS = static_cast<unsigned long long>(S < 0 ? -S : S);
            const unsigned __int128 d = Q * static_cast<unsigned>(cnt) - static_cast<unsigned __int128>(absS) * absS;   // n Q - S^2 >= 0
            const double dd = ldexp(static_cast<double>(static_cast<unsigned long long>(d >> 64)), 64) +
                              static_cast<double>(static_cast<unsigned long long>(d));
            // sum (r - mean)^2 = (n Q - S^2) / n in grid units^2 = (n Q - S^2) * n * unit^2
            sigma = sqrt(dd * static_cast<double>(cnt) * unit * unit / static_cast<double>(dof));
        }
    };
    double mean, sigma, unit;
    int cnt, shift;
    if (i < n_seg && (a.seg_mean != nullptr || a.seg_std != nullptr)) {
        stats(i, mean, sigma, unit, cnt, shift);
        if (a.seg_mean) a.seg_mean[i] = static_cast<float>(mean);
        if (a.seg_std) a.seg_std[i] = static_cast<float>(sigma);
    }
    if (i < a.n_inv) {
        const int seg = a.seg_scratch[i];
        float adv = 0.f;
        if (seg >= 0) {
            stats(seg, mean, sigma, unit, cnt, shift);
            const double denom = sigma + static_cast<double>(a.eps);
            if (cnt - a.ddof > 0 && denom != 0.0 && unit != 0.0) {
                const long long e = static_cast<long long>(cnt) * seg_quantise(a.r_scratch[i], shift) - __ldcg(&t.sum[seg]);
                adv = static_cast<float>(static_cast<double>(e) * unit / denom);
            }
        }
        a.adv_inv[i] = adv;
    }
}

// All blocks of a cooperative launch meet: counter reaches `target`.  Bounded: on expiry the timeout status is set and
// the block goes on (the call's results are then undefined, the host sees UNITY_ERR_TIMEOUT).
__device__ __forceinline__ void adv_grid_barrier(const AdvArgs& a, unsigned target) {
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned* counter = reinterpret_cast<unsigned*>(a.seg_table);
        __threadfence();
        atomicAdd(counter, 1u);
        const long long t0 = clock64();
        bool ok = true;
        while (*reinterpret_cast<volatile unsigned*>(counter) < target) {
            if (clock64() - t0 > 2000000000LL) { ok = false; break; }
        }
        if (!ok) atomicOr(a.status, kStatusTimeout);
        __threadfence();
    }
    __syncthreads();
}

// phase 0: all three passes with grid barriers (cooperative launch); 1, 2, 3: one pass (plain launches)
__global__ void k_adv_stats(AdvArgs a, int phase) {
    const int n_fin = max(a.n_inv, a.n_groups * a.n_roles);
    const int stride = gridDim.x * blockDim.x, first = blockIdx.x * blockDim.x + threadIdx.x;
    if (phase == 0 || phase == 1)
        for (int s = first; s < a.n_inv; s += stride) adv_pass_combine(a, s);
    if (phase == 0) adv_grid_barrier(a, gridDim.x);
    if (phase == 0 || phase == 2)
        for (int s = first; s < a.n_inv; s += stride) adv_pass_sums(a, s);
    if (phase == 0) adv_grid_barrier(a, 2u * gridDim.x);
    if (phase == 0 || phase == 3)
        for (int i = first; i < n_fin; i += stride) adv_pass_finish(a, i);
}

// A block broadcasts rounds x 1024 tokens; in a round each thread handles four consecutive tokens (one 32-bit mask
// load, one 128-bit store), so every warp instruction covers 128 B of mask and 512 B of output contiguously.
// The owning invocation is found by binary search once per thread (a chain of dependent loads, amortised over the
// rounds) and advanced linearly afterwards.
__global__ void k_adv_broadcast(AdvArgs a, int rounds) {
    const long long block0 = static_cast<long long>(blockIdx.x) * (blockDim.x * 4) * rounds;
    const bool mask_al = (reinterpret_cast<uintptr_t>(a.tok_mask) & 3) == 0;
    const bool out_al = (reinterpret_cast<uintptr_t>(a.adv_tok) & 15) == 0;
    int s = -1;
    long long end = 0;
    float adv = 0.f;
    for (int round = 0; round < rounds; ++round) {
        const long long i0 = block0 + (static_cast<long long>(round) * blockDim.x + threadIdx.x) * 4;
        if (i0 >= a.n_tok) return;
        if (s < 0) {
            s = find_invocation(a.cu_seqlens, a.n_inv, i0);
            end = a.cu_seqlens[s + 1];
            adv = a.adv_inv[s];
        }
        float out[4];
        const int n = static_cast<int>(min(4LL, a.n_tok - i0));
        unsigned m4 = 0x01010101u;
        if (a.tok_mask) {
            if (n == 4 && mask_al) m4 = *reinterpret_cast<const unsigned*>(a.tok_mask + i0);
            else { m4 = 0; for (int j = 0; j < n; ++j) m4 |= static_cast<unsigned>(a.tok_mask[i0 + j]) << (8 * j); }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const long long i = i0 + j;
            if (j < n) {
                while (i >= end && s + 1 < a.n_inv) { ++s; end = a.cu_seqlens[s + 1]; adv = a.adv_inv[s]; }
                out[j] = ((m4 >> (8 * j)) & 0xffu) ? adv : 0.f;
            } else out[j] = 0.f;
        }
        if (n == 4 && out_al) *reinterpret_cast<float4*>(a.adv_tok + i0) = make_float4(out[0], out[1], out[2], out[3]);
        else for (int j = 0; j < n; ++j) a.adv_tok[i0 + j] = out[j];
    }
}

// The same broadcast with one warp per invocation, for batches of long invocations: no search; after the tokens up to
// the next multiple of 4, the warp walks the invocation 512 tokens per step: four times, every lane loads the four
// mask bytes of its quad of tokens (128 B contiguous per warp) and stores one 128-bit vector (512 B contiguous per
// warp), all four loads issued before the first store.
__global__ void k_adv_broadcast_inv(AdvArgs a) {
    const int s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (s >= a.n_inv) return;
    const long long lo = a.cu_seqlens[s], hi = a.cu_seqlens[s + 1];
    const float adv = a.adv_inv[s];
    const long long head_end = min(hi, (lo + 3) & ~3LL);
    for (long long i = lo + lane; i < head_end; i += 32) a.adv_tok[i] = (a.tok_mask == nullptr || a.tok_mask[i]) ? adv : 0.f;
    const long long n_quad = (hi - head_end) >> 2;
    for (long long q0 = 0; q0 < n_quad; q0 += 128) {
        unsigned m[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long q = q0 + u * 32 + lane;
            m[u] = 0x01010101u;
            if (a.tok_mask != nullptr && q < n_quad) m[u] = *reinterpret_cast<const unsigned*>(a.tok_mask + head_end + (q << 2));
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long q = q0 + u * 32 + lane;
            if (q < n_quad)
                *reinterpret_cast<float4*>(a.adv_tok + head_end + (q << 2)) =
                    make_float4((m[u] & 0xffu) ? adv : 0.f, (m[u] & 0xff00u) ? adv : 0.f, (m[u] & 0xff0000u) ? adv : 0.f,
                                (m[u] & 0xff000000u) ? adv : 0.f);
        }
    }
    for (long long i = head_end + (n_quad << 2) + lane; i < hi; i += 32)
        a.adv_tok[i] = (a.tok_mask == nullptr || a.tok_mask[i]) ? adv : 0.f;
}

// ------------------------------------------------------------------------------------------------
// Routing: stable partition of the valid tokens by model id (count, scan, assign)
// ------------------------------------------------------------------------------------------------
__global__ void k_route_count(RouteArgs a) {
    __shared__ int cnt[UNITY_MAX_MODELS];
    if (threadIdx.x < UNITY_MAX_MODELS) cnt[threadIdx.x] = 0;
    __syncthreads();
    const long long i = static_cast<long long>(blockIdx.x) * kRouteBlock + threadIdx.x;
    if (i < a.n_tok) {
        int model = -1;
        const bool on = a.tok_mask ? (a.tok_mask[i] != 0) : true;
        if (on) {
            const int s = find_invocation(a.cu_seqlens, a.n_inv, i);
            const int role = a.inv_role[s];
            const int tgt = a.target[i];
            if (role >= 0 && role < a.n_roles && tgt >= 0 && tgt < a.V) {
                model = a.role_model[role];
                if (model < 0 || model >= a.K) model = -1;
            }
            if (model < 0) atomicOr(a.status, kStatusBadIndex);
            else atomicAdd(&cnt[model], 1);
        }
        a.tok_model[i] = static_cast<int8_t>(model);
    }
    __syncthreads();
    if (threadIdx.x < a.K) a.blk_cnt[blockIdx.x * a.K + threadIdx.x] = cnt[threadIdx.x];
}

// One block: exclusive scan of the per-block counts of each model; then slot offsets padded to the row tile.
__global__ void k_route_scan(RouteArgs a) {
    __shared__ int part[1024];
    __shared__ int total[UNITY_MAX_MODELS];
    const int tid = threadIdx.x, nt = blockDim.x;
    const int per = (a.n_blocks + nt - 1) / nt;
    const int b0 = tid * per, b1 = min(b0 + per, a.n_blocks);
    for (int k = 0; k < a.K; ++k) {
        int s = 0;
        for (int b = b0; b < b1; ++b) s += a.blk_cnt[b * a.K + k];
        part[tid] = s;
        __syncthreads();
        for (int off = 1; off < nt; off <<= 1) {     // inclusive Hillis-Steele scan of the thread sums
            const int v = (tid >= off) ? part[tid - off] : 0;
            __syncthreads();
            part[tid] += v;
            __syncthreads();
        }
        int run = part[tid] - s;
        if (tid == nt - 1) total[k] = part[tid];
        for (int b = b0; b < b1; ++b) { const int c = a.blk_cnt[b * a.K + k]; a.blk_cnt[b * a.K + k] = run; run += c; }
        __syncthreads();
    }
    if (tid == 0) {
        int off = 0;
        long long sbase = 0;
        for (int k = 0; k < a.K; ++k) {
            const int rows = (total[k] + kTileM - 1) / kTileM * kTileM;
            a.plan->counts[k] = total[k];
            a.plan->off[k] = off;
            a.plan->stats_base[k] = sbase;
            off += rows;
            sbase += rows > 0 ? forward_shape(a.fwd, rows).stats_rows : 0;
        }
        a.plan->off[a.K] = off;
    }
}

__global__ void k_route_assign(RouteArgs a) {
    __shared__ int warp_cnt[kRouteBlock / 32][UNITY_MAX_MODELS];
    const long long i = static_cast<long long>(blockIdx.x) * kRouteBlock + threadIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int model = (i < a.n_tok) ? a.tok_model[i] : -1;
    int rank = 0;
    for (int k = 0; k < a.K; ++k) {
        const unsigned bal = __ballot_sync(kFull, model == k);
        if (model == k) rank = __popc(bal & ((1u << lane) - 1u));
        if (lane == 0) warp_cnt[warp][k] = __popc(bal);
    }
    __syncthreads();
    if (i >= a.n_tok) return;
    if (model < 0) { a.tok_slot[i] = -1; return; }
    int before = 0;
    for (int w = 0; w < warp; ++w) before += warp_cnt[w][model];
    const int slot = a.plan->off[model] + a.blk_cnt[blockIdx.x * a.K + model] + before + rank;
    a.tok_slot[i] = slot;
    a.slot_tok[slot] = static_cast<int>(i);
}

// One warp per packed row: 128-bit copies of the hidden row (zeros for padding slots).
__global__ void k_gather_rows(const __nv_bfloat16* __restrict__ hidden, const int32_t* __restrict__ target,
                              const int* __restrict__ slot_tok, const DevPlan* __restrict__ plan, int K, int H,
                              __nv_bfloat16* __restrict__ hp, int* __restrict__ target_p) {
    const long long slot = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (slot >= plan->off[K]) return;
    const int tok = slot_tok[slot];
    const int n16 = H >> 3;
    uint4* dst = reinterpret_cast<uint4*>(hp + static_cast<long long>(slot) * H);
    if (tok >= 0) {
        const uint4* src = reinterpret_cast<const uint4*>(hidden + static_cast<long long>(tok) * H);
        for (int j = lane; j < n16; j += 32) dst[j] = src[j];
    } else {
        for (int j = lane; j < n16; j += 32) dst[j] = make_uint4(0, 0, 0, 0);
    }
    if (lane == 0) target_p[slot] = tok >= 0 ? target[tok] : 0;
}

// ------------------------------------------------------------------------------------------------
// Per-token PPO terms
// ------------------------------------------------------------------------------------------------
struct PpoTerms {
    float rho, pg, kl, tok_loss, dl_dlogp, clipped;
};
__device__ __forceinline__ PpoTerms ppo_terms(float logp, float ent, float old_lp, float ref_lp, float adv,
                                              float clip_lo, float clip_hi, float kl_coef, int kl_mode,
                                              float ent_coef) {
    PpoTerms t;
    t.rho = expf(logp - old_lp);
    const float rho_c = fminf(fmaxf(t.rho, 1.f - clip_lo), 1.f + clip_hi);
    const float unclipped = -t.rho * adv, clipped = -rho_c * adv;
    const bool u = unclipped >= clipped;     // ties take the unclipped branch
    t.pg = u ? unclipped : clipped;
    t.clipped = u ? 0.f : 1.f;
    const float d = ref_lp - logp;
    float dkl;
    if (kl_mode == 1) { t.kl = -d; dkl = 1.f; }
    else if (kl_mode == 2) { t.kl = 0.5f * d * d; dkl = -d; }
    else { const float e = expm1f(d); t.kl = e - d; dkl = -e; }
    t.tok_loss = t.pg + kl_coef * t.kl - ent_coef * ent;
    t.dl_dlogp = (u ? -adv * t.rho : 0.f) + kl_coef * dkl;
    return t;
}

// One thread per packed row: merge the vocabulary splits, form lse / entropy / logp, then the loss terms.
__global__ void k_finish_rows(TokenArgs a, int with_loss) {
    // Where the statistics of a row lie follows from the shape of the forward launch that wrote them, and that from the
    // rows the launch covered: one block of one model's rows, or each model's whole range.
    __shared__ FwdShape sh_shape[UNITY_MAX_MODELS];
    __shared__ int sh_first[UNITY_MAX_MODELS], sh_rows[UNITY_MAX_MODELS];
    __shared__ long long sh_base[UNITY_MAX_MODELS];
    __shared__ int sh_lo, sh_hi;
    if (threadIdx.x < UNITY_MAX_MODELS) {
        const int k = threadIdx.x;
        int first = 0, rows = 0;
        long long base = 0;
        if (k < a.K) {
            if (a.block.model >= 0) {
                if (k == a.block.model) span_resolve(a.block, first, rows);
            } else {
                first = a.plan->off[k];
                rows = a.plan->off[k + 1] - first;
                base = a.plan->stats_base[k];
            }
        }
        sh_first[k] = first; sh_rows[k] = rows; sh_base[k] = base;
        if (rows > 0 && a.lse_in == nullptr) sh_shape[k] = forward_shape(a.fwd, rows);
        if (k == 0) {
            if (a.block.model >= 0) { int f, r; span_resolve(a.block, f, r); sh_lo = f; sh_hi = f + r; }
            else { sh_lo = 0; sh_hi = a.plan->off[a.K]; }
        }
    }
    __syncthreads();
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= sh_hi - sh_lo) return;
    const int slot = sh_lo + static_cast<int>(idx);
    const int tok = a.slot_tok[slot];
    if (tok < 0) {
        a.row_lse[slot] = 0.f; a.row_ent[slot] = 0.f; a.row_logp[slot] = 0.f;
        if (with_loss) { a.coef_a[slot] = 0.f; a.coef_b[slot] = 0.f; }
        return;
    }
    const int k = a.tok_model[tok];
    float lse, ent, logp;
    if (a.lse_in) {
        // the caller already evaluated this policy on these rows (unity_logprob_fwd): no forward sweep was run
        lse = a.lse_in[tok]; ent = a.entropy_in[tok]; logp = a.logp_in[tok];
    } else {
        const FwdShape& fs = sh_shape[k];
        long long pitch = sh_rows[k];
        const int r = slot - sh_first[k];
        const float4* st = a.stats + sh_base[k] + r;
        int n_splits = fs.splits;
        const long long last_row0 = static_cast<long long>(fs.last_m0) * a.fwd.tile_rows;
        if (r >= last_row0) {                                 // swept in the launch's short last round
            st = a.stats + sh_base[k] + static_cast<long long>(fs.splits) * pitch + (r - last_row0);
            pitch -= last_row0;
            n_splits = fs.last_splits;
        }
        const float c = a.scale * 1.4426950408889634f;    // exp(scale*x) = exp2(c*x)
        float m = -3.0e38f;
        for (int j = 0; j < n_splits; ++j) m = fmaxf(m, st[j * pitch].x);
        float s = 0.f, t = 0.f, zy = -3.0e38f;
        for (int j = 0; j < n_splits; ++j) {
            const float4 p = st[j * pitch];
            const float w = exp2f((p.x - m) * c);
            s += p.y * w;
            t += p.z * w;
            zy = fmaxf(zy, p.w);
        }
        lse = a.scale * m + logf(s);
        ent = lse - a.scale * (t / s);
        logp = a.scale * zy - lse;
    }
    a.row_lse[slot] = lse; a.row_ent[slot] = ent; a.row_logp[slot] = logp;
    if (a.logp) a.logp[tok] = logp;
    if (a.entropy) a.entropy[tok] = ent;
    if (a.lse) a.lse[tok] = lse;
    if (!with_loss) return;
    const float Mk = a.has_norm ? a.norm[k] : fmaxf(static_cast<float>(a.plan->counts[k]), 1.f);
    const PpoTerms p = ppo_terms(logp, ent, a.old_logp[tok], a.ref_logp[tok], a.adv_tok[tok], a.clip_lo, a.clip_hi,
                                 a.kl_coef, a.kl_mode, a.ent_coef);
    a.coef_a[slot] = a.scale * (p.dl_dlogp / Mk);
    a.coef_b[slot] = a.scale * (-a.ent_coef / Mk);
    if (a.tok_loss) a.tok_loss[tok] = p.tok_loss;
}

// One warp per invocation: nine sums over its valid tokens in a fixed order.
__global__ void k_inv_reduce(TokenArgs a) {
    const int s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (s >= a.n_inv) return;
    float acc[9];
#pragma unroll
    for (int j = 0; j < 9; ++j) acc[j] = 0.f;
    const long long lo = a.cu_seqlens[s], hi = a.cu_seqlens[s + 1];
    for (long long i = lo + lane; i < hi; i += 32) {
        const int slot = a.tok_slot[i];
        if (slot < 0) continue;
        const float logp = a.row_logp[slot], ent = a.row_ent[slot], adv = a.adv_tok[i];
        const PpoTerms p = ppo_terms(logp, ent, a.old_logp[i], a.ref_logp[i], adv, a.clip_lo, a.clip_hi, a.kl_coef,
                                     a.kl_mode, a.ent_coef);
        acc[0] += 1.f; acc[1] += p.pg; acc[2] += p.kl; acc[3] += ent; acc[4] += p.clipped; acc[5] += p.rho;
        acc[6] += logp; acc[7] += adv; acc[8] += p.tok_loss;
    }
#pragma unroll
    for (int j = 0; j < 9; ++j) acc[j] = warp_sum(acc[j]);
    if (lane == 0)
        for (int j = 0; j < 9; ++j) a.inv_sums[s * 9 + j] = acc[j];
}

// One warp per class (K models, then n_roles roles): fixed-order sum over the invocations of the class.
__global__ void k_class_reduce(TokenArgs a) {
    const int c = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (c >= a.K + a.n_roles) return;
    float acc[9];
#pragma unroll
    for (int j = 0; j < 9; ++j) acc[j] = 0.f;
    for (int s = lane; s < a.n_inv; s += 32) {
        const int role = a.inv_role[s];
        if (role < 0 || role >= a.n_roles) continue;
        const bool mine = (c < a.K) ? (a.role_model[role] == c) : (role == c - a.K);
        if (!mine) continue;
#pragma unroll
        for (int j = 0; j < 9; ++j) acc[j] += a.inv_sums[s * 9 + j];
    }
#pragma unroll
    for (int j = 0; j < 9; ++j) acc[j] = warp_sum(acc[j]);
    if (lane != 0) return;
    const float dn = fmaxf(acc[0], 1.f);
    if (a.metrics) {
        float* m = a.metrics + c * UNITY_N_METRICS;
        m[0] = acc[0];
        for (int j = 1; j < 8; ++j) m[j] = acc[j] / dn;
    }
    if (c < a.K) a.loss[c] = acc[8] / (a.has_norm ? a.norm[c] : fmaxf(static_cast<float>(a.plan->counts[c]), 1.f));
}

// Stashed logits -> logit gradients, in place.  A block converts 8192 consecutive columns of one row: every thread
// first issues its four 128-bit loads (4 KiB apart, so each warp access covers 512 contiguous bytes), then converts
// and stores them.  Streaming: 2 B read + 2 B written per logit.
constexpr int kGradVecs = 4;
__global__ void __launch_bounds__(256) k_logit_grad_inplace(LogitGradArgs a) {
    const int c_first = blockIdx.x * (256 * 8 * kGradVecs) + threadIdx.x * 8;
    int row0, rows;
    span_resolve(a.span, row0, rows);
    for (int r = blockIdx.y; r < rows; r += gridDim.y) {
        const int slot = row0 + r;
        uint4* row = reinterpret_cast<uint4*>(a.Z + static_cast<long long>(r) * a.ld);
        uint4 raw[kGradVecs];
#pragma unroll
        for (int u = 0; u < kGradVecs; ++u) {
            const int c0 = c_first + u * 2048;
            if (c0 < a.cols) raw[u] = row[c0 >> 3];
        }
        const float ca = a.coef_a[slot], cb = a.coef_b[slot], lse = a.row_lse[slot];
        const float hl = a.row_ent[slot] - lse;
        const int tgt = a.target_p[slot] - a.vocab0;
        const float shift = -lse * 1.4426950408889634f;
#pragma unroll
        for (int u = 0; u < kGradVecs; ++u) {
            const int c0 = c_first + u * 2048;
            if (c0 >= a.cols) continue;
            __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&raw[u]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 z = __bfloat1622float2(h2[j]);
                const float p0 = exp2f(fmaf(z.x, 1.4426950408889634f, shift));
                const float p1 = exp2f(fmaf(z.y, 1.4426950408889634f, shift));
                float g0 = -p0 * fmaf(cb, z.x + hl, ca), g1 = -p1 * fmaf(cb, z.y + hl, ca);
                if (c0 + 2 * j == tgt) g0 += ca;
                if (c0 + 2 * j + 1 == tgt) g1 += ca;
                h2[j] = __floats2bfloat162_rn(g0, g1);
            }
            row[c0 >> 3] = raw[u];
        }
    }
}

__global__ void k_zero_masked_rows(const int* __restrict__ tok_slot, long long n_tok, int H,
                                   __nv_bfloat16* __restrict__ dHidden) {
    const long long tok = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (tok >= n_tok || tok_slot[tok] >= 0) return;
    uint4* dst = reinterpret_cast<uint4*>(dHidden + tok * H);
    for (int j = lane; j < (H >> 3); j += 32) dst[j] = make_uint4(0, 0, 0, 0);
}

// dst[0, n4) = 0 (128-bit stores, grid-stride) when model k has no valid row; returns at once otherwise.
__global__ void k_zero_if_empty(float4* __restrict__ dst, long long n4, const DevPlan* __restrict__ plan, int k) {
    if (plan->counts[k] != 0) return;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n4; i += stride)
        dst[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

__global__ void k_store_dhidden(const float* __restrict__ dHc, const int* __restrict__ slot_tok, RowSpan span,
                                int H, __nv_bfloat16* __restrict__ dHidden) {
    const int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    int slot0, n_rows;
    span_resolve(span, slot0, n_rows);
    if (r >= n_rows) return;
    const int tok = slot_tok[slot0 + r];
    if (tok < 0) return;
    const float4* src = reinterpret_cast<const float4*>(dHc + static_cast<long long>(r) * H);
    uint2* dst = reinterpret_cast<uint2*>(dHidden + static_cast<long long>(tok) * H);
    for (int j = lane; j < (H >> 2); j += 32) {
        const float4 v = src[j];
        __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
        uint2 o;
        o.x = *reinterpret_cast<unsigned*>(&lo);
        o.y = *reinterpret_cast<unsigned*>(&hi);
        dst[j] = o;
    }
}

// ------------------------------------------------------------------------------------------------
// Token-level generalized advantage estimation: one warp per sequence, walking it backwards 32 tokens at a time.
// Inside a chunk the recurrence A_t = delta_t + c*A_next is a composition of affine maps x -> b + a*x, evaluated
// with a suffix scan over the lanes (masked tokens are the identity map); the value of the next unmasked token
// comes from a ballot.  Loads and stores are 128-byte coalesced per warp.
struct GaeArgs {
    int n_inv;
    const int64_t* cu_seqlens;
    const float *rewards, *values;
    const uint8_t* tok_mask;
    float gamma, lam;
    float *adv, *ret;
};

__global__ void k_gae(GaeArgs a) {
    const int s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (s >= a.n_inv) return;
    const long long lo = a.cu_seqlens[s], hi = a.cu_seqlens[s + 1];
    const float c = a.gamma * a.lam;
    float carry_adv = 0.f, carry_val = 0.f;       // A and V of the next unmasked token (0 past the end)
    for (long long c0 = hi - 32; c0 > lo - 32; c0 -= 32) {
        const long long t = c0 + lane;
        const bool in = t >= lo && t < hi;
        const bool on = in && (a.tok_mask ? a.tok_mask[t] != 0 : true);
        const float v = on ? a.values[t] : 0.f;
        const float r = on ? a.rewards[t] : 0.f;
        const unsigned valid = __ballot_sync(kFull, on);
        const unsigned above = lane == 31 ? 0u : (valid & (0xffffffffu << (lane + 1)));
        const int j = above ? __ffs(above) - 1 : 0;
        const float v_peer = __shfl_sync(kFull, v, j);
        const float v_next = above ? v_peer : carry_val;
        const float delta = r + a.gamma * v_next - v;
        // suffix scan of the maps (ma, mb): result on lane i is the composition of lanes i, i+1, ..., 31
        float ma = on ? c : 1.f, mb = on ? delta : 0.f;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float pa = __shfl_down_sync(kFull, ma, o), pb = __shfl_down_sync(kFull, mb, o);
            if (lane + o < 32) { mb = fmaf(ma, pb, mb); ma = ma * pa; }
        }
        const float adv = fmaf(ma, carry_adv, mb);
        if (in) {
            a.adv[t] = on ? adv : 0.f;
            a.ret[t] = on ? adv + v : 0.f;
        }
        carry_adv = __shfl_sync(kFull, adv, 0);    // lane 0 holds the composition of the whole chunk
        if (valid) carry_val = __shfl_sync(kFull, v, __ffs(valid) - 1);
    }
}

// The same recurrence with four tokens per lane (128 tokens per warp step, 128-bit accesses; chunks are aligned to
// absolute token indices that are multiples of 128, tokens outside the sequence count as masked).  Inside a lane the
// four maps are composed one after the other; across lanes by the suffix scan; then every token's advantage follows
// from the advantage entering its lane.
__global__ void k_gae_vec(GaeArgs a) {
    const int s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (s >= a.n_inv) return;
    const long long lo = a.cu_seqlens[s], hi = a.cu_seqlens[s + 1];
    if (hi <= lo) return;
    const float c = a.gamma * a.lam;
    float carry_adv = 0.f, carry_val = 0.f;
    for (long long c0 = ((hi - 1) >> 7) << 7; c0 + 128 > lo; c0 -= 128) {
        const long long t0 = c0 + 4 * lane;
        float v[4] = {0.f, 0.f, 0.f, 0.f}, r[4] = {0.f, 0.f, 0.f, 0.f};
        unsigned m4 = 0u;
        const bool whole = t0 >= lo && t0 + 4 <= hi;
        if (whole) {
            const float4 vv = *reinterpret_cast<const float4*>(a.values + t0);
            const float4 rr = *reinterpret_cast<const float4*>(a.rewards + t0);
            v[0] = vv.x; v[1] = vv.y; v[2] = vv.z; v[3] = vv.w;
            r[0] = rr.x; r[1] = rr.y; r[2] = rr.z; r[3] = rr.w;
            m4 = a.tok_mask ? *reinterpret_cast<const unsigned*>(a.tok_mask + t0) : 0x01010101u;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long t = t0 + j;
                if (t >= lo && t < hi) {
                    v[j] = a.values[t]; r[j] = a.rewards[t];
                    if (a.tok_mask ? a.tok_mask[t] != 0 : true) m4 |= 0x01u << (8 * j);
                }
            }
        }
        bool on[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) on[j] = ((m4 >> (8 * j)) & 0xffu) != 0;
        const bool any = m4 != 0u;
        // value of the first unmasked token of the lanes above (or of the chunks above)
        float first_v = 0.f;
#pragma unroll
        for (int j = 3; j >= 0; --j) if (on[j]) first_v = v[j];
        const unsigned valid = __ballot_sync(kFull, any);
        const unsigned above = lane == 31 ? 0u : (valid & (0xffffffffu << (lane + 1)));
        const float v_peer = __shfl_sync(kFull, first_v, above ? __ffs(above) - 1 : 0);
        float v_next = above ? v_peer : carry_val;
        // the lane's tokens from the last to the first: token j maps the advantage entering the lane, x, to pb[j] + pa[j]*x
        float pa[4], pb[4];
        float ma = 1.f, mb = 0.f;
#pragma unroll
        for (int j = 3; j >= 0; --j) {
            if (on[j]) {
                const float delta = r[j] + a.gamma * v_next - v[j];
                mb = fmaf(c, mb, delta);
                ma = ma * c;
                v_next = v[j];
            }
            pa[j] = ma; pb[j] = mb;
        }
        // suffix scan of the lane maps: lane i ends with the composition of lanes i .. 31
        float sa = ma, sb = mb;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float qa = __shfl_down_sync(kFull, sa, o), qb = __shfl_down_sync(kFull, sb, o);
            if (lane + o < 32) { sb = fmaf(sa, qb, sb); sa = sa * qa; }
        }
        const float at_lane = fmaf(sa, carry_adv, sb);            // advantage at this lane's first unmasked token
        const float from_above = __shfl_down_sync(kFull, at_lane, 1);
        const float x = lane == 31 ? carry_adv : from_above;      // advantage entering this lane
        float adv[4], ret[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            adv[j] = on[j] ? fmaf(pa[j], x, pb[j]) : 0.f;
            ret[j] = on[j] ? adv[j] + v[j] : 0.f;
        }
        if (whole) {
            *reinterpret_cast<float4*>(a.adv + t0) = make_float4(adv[0], adv[1], adv[2], adv[3]);
            *reinterpret_cast<float4*>(a.ret + t0) = make_float4(ret[0], ret[1], ret[2], ret[3]);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long t = t0 + j;
                if (t >= lo && t < hi) { a.adv[t] = adv[j]; a.ret[t] = ret[j]; }
            }
        }
        carry_adv = __shfl_sync(kFull, at_lane, 0);
        if (valid) carry_val = __shfl_sync(kFull, first_v, __ffs(valid) - 1);
    }
}

// ------------------------------------------------------------------------------------------------
// Turn-level reward assembly: one thread per invocation gathers its trajectory's score(s).
__global__ void k_reward_assembly(RewardArgs a) {
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= a.n_inv) return;
    float out = 0.f;
    const int v = a.inv_role[s], j = a.inv_traj[s];
    if (v < 0 || v >= a.n_roles || j < 0 || j >= a.n_traj) {
        atomicOr(a.status, kStatusBadIndex);
    } else {
        const int mode = a.mode[v];
        const int u = a.inv_turn[s] + a.shift[v];
        const int n = min(a.n_scores ? a.n_scores[j] : a.max_turns, a.max_turns);
        const bool ended = a.inv_end ? a.inv_end[s] != 0 : false;
        if (mode != 0 && u >= 0 && u < n && !ended) {
            const float* sc = a.score + static_cast<long long>(j) * a.max_turns;
            out = mode == 1 ? sc[u] : sc[u] - (u >= 1 ? sc[u - 1] : 0.f);
        }
    }
    a.r_turn[s] = out;
}

// ------------------------------------------------------------------------------------------------
// Critic update: clipped value loss.  The token data is read once: a first pass over the mask bytes alone gives the
// denominators M_k, the main pass then forms loss terms and gradients; all sums have a fixed order.
struct ValueTerm {
    float loss, grad, clipped;
};
__device__ __forceinline__ ValueTerm value_term(float v, float ov, float ret, float clip_v) {
    const float d = v - ov;
    // inside the range the clipped estimate IS v; outside it is the end of the range
    const float vc = fabsf(d) <= clip_v ? v : ov + copysignf(clip_v, d);
    const float eu = v - ret, ec = vc - ret;
    const float su = eu * eu, sc = ec * ec;
    const bool unclipped = su >= sc;            // ties take the unclipped branch
    ValueTerm t;
    t.loss = 0.5f * (unclipped ? su : sc);
    t.grad = unclipped ? eu : 0.f;
    t.clipped = unclipped ? 0.f : 1.f;
    return t;
}

// Denominator of model k: the caller's norm, else the valid tokens counted by k_value_count (at least 1).
__device__ __forceinline__ float value_Mk(const ValueArgs& a, int k) {
    return a.has_norm ? a.norm[k] : fmaxf(static_cast<float>(a.model_cnt[k]), 1.f);
}

// (1) valid tokens per invocation (mask bytes only) and per model.  The per-model totals are integers added with atomics
// (one per block and model): exact and independent of the order in which the blocks arrive.
__global__ void k_value_count(ValueArgs a) {
    __shared__ int block_cnt[UNITY_MAX_MODELS];
    if (threadIdx.x < UNITY_MAX_MODELS) block_cnt[threadIdx.x] = 0;
    __syncthreads();
    const int s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (s < a.n_inv) {
        const int role = a.inv_role[s];
        const bool role_ok = role >= 0 && role < a.n_roles && a.role_model[role] >= 0 && a.role_model[role] < a.K;
        const long long lo = a.cu_seqlens[s], hi = a.cu_seqlens[s + 1];
        int cnt = 0;
        if (role_ok) {
            if (a.tok_mask == nullptr) {
                cnt = lane == 0 ? static_cast<int>(hi - lo) : 0;
            } else {
                // bytes up to the next 16-byte boundary one by one, then 16 mask bytes per lane and load, then the rest
                const uintptr_t addr = reinterpret_cast<uintptr_t>(a.tok_mask) + static_cast<uintptr_t>(lo);
                const long long head_end = min(hi, lo + static_cast<long long>((16 - (addr & 15)) & 15));
                for (long long i = lo + lane; i < head_end; i += 32) cnt += a.tok_mask[i] != 0;
                const long long n_vec = (hi - head_end) >> 4;
                const uint4* mv = reinterpret_cast<const uint4*>(a.tok_mask + head_end);
                for (long long q = lane; q < n_vec; q += 32) {
                    const uint4 m = mv[q];
                    cnt += (__popc(__vcmpne4(m.x, 0u)) + __popc(__vcmpne4(m.y, 0u)) + __popc(__vcmpne4(m.z, 0u)) +
                            __popc(__vcmpne4(m.w, 0u))) >> 3;
                }
                for (long long i = head_end + (n_vec << 4) + lane; i < hi; i += 32) cnt += a.tok_mask[i] != 0;
            }
        }
        cnt = warp_sum_int(cnt);
        if (lane == 0) {
            if (!role_ok && hi > lo) atomicOr(a.status, kStatusBadIndex);
            a.inv_sums[s * 3 + 0] = static_cast<float>(cnt);
            if (role_ok && cnt > 0) atomicAdd(&block_cnt[a.role_model[role]], cnt);
        }
    }
    __syncthreads();
    if (threadIdx.x < a.K && block_cnt[threadIdx.x] > 0)
        atomicAdd(&a.model_cnt[threadIdx.x], static_cast<unsigned long long>(block_cnt[threadIdx.x]));
}

// Fixed-order sum over the 1024 threads of a block: lanes, then the 32 warp totals.
__device__ __forceinline__ float block_sum_1024(float v, float* sh) {
    v = warp_sum(v);
    __syncthreads();                                   // sh may still be read from an earlier call
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
    if (threadIdx.x < 32) t = warp_sum(sh[threadIdx.x]);
    return t;                                          // valid in warp 0
}

// (3) the one pass over the token data: loss terms, gradient (already divided by M_k), per-invocation sums.
__global__ void k_value_main(ValueArgs a) {
    const int s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (s >= a.n_inv) return;
    const int role = a.inv_role[s];
    const bool role_ok = role >= 0 && role < a.n_roles && a.role_model[role] >= 0 && a.role_model[role] < a.K;
    const float inv_M = 1.f / (role_ok ? value_Mk(a, a.role_model[role]) : 1.f);
    const long long lo = a.cu_seqlens[s], hi = a.cu_seqlens[s + 1];
    float sum = 0.f, clp = 0.f;
    auto one = [&](long long i) {
        const bool on = role_ok && (a.tok_mask ? a.tok_mask[i] != 0 : true);
        float l = 0.f, gr = 0.f;
        if (on) {
            const ValueTerm t = value_term(a.values[i], a.old_values[i], a.returns[i], a.clip_v);
            l = t.loss; gr = t.grad * inv_M; sum += t.loss; clp += t.clipped;
        }
        a.dvalues[i] = gr;
        if (a.tok_loss) a.tok_loss[i] = l;
    };
    if (!a.vec_ok) {
        for (long long i = lo + lane; i < hi; i += 32) one(i);
    } else {
        // tokens up to a multiple of four one by one, then four tokens per lane with 128-bit accesses, then the rest
        const long long head_end = min(hi, (lo + 3) & ~3LL);
        for (long long i = lo + lane; i < head_end; i += 32) one(i);
        const long long n_quad = (hi - head_end) >> 2;
        for (long long q = lane; q < n_quad; q += 32) {
            const long long i = head_end + (q << 2);
            const float4 v = *reinterpret_cast<const float4*>(a.values + i);
            const float4 ov = *reinterpret_cast<const float4*>(a.old_values + i);
            const float4 rt = *reinterpret_cast<const float4*>(a.returns + i);
            const unsigned m4 = a.tok_mask ? *reinterpret_cast<const unsigned*>(a.tok_mask + i) : 0x01010101u;
            const float vv[4] = {v.x, v.y, v.z, v.w}, oo[4] = {ov.x, ov.y, ov.z, ov.w}, rr[4] = {rt.x, rt.y, rt.z, rt.w};
            float g4[4], l4[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                g4[j] = 0.f; l4[j] = 0.f;
                if (role_ok && ((m4 >> (8 * j)) & 0xffu)) {
                    const ValueTerm t = value_term(vv[j], oo[j], rr[j], a.clip_v);
                    l4[j] = t.loss; g4[j] = t.grad * inv_M; sum += t.loss; clp += t.clipped;
                }
            }
            *reinterpret_cast<float4*>(a.dvalues + i) = make_float4(g4[0], g4[1], g4[2], g4[3]);
            if (a.tok_loss) *reinterpret_cast<float4*>(a.tok_loss + i) = make_float4(l4[0], l4[1], l4[2], l4[3]);
        }
        for (long long i = head_end + (n_quad << 2) + lane; i < hi; i += 32) one(i);
    }
    sum = warp_sum(sum); clp = warp_sum(clp);
    if (lane == 0) { a.inv_sums[s * 3 + 1] = sum; a.inv_sums[s * 3 + 2] = clp; }
}

// (4) loss and clip fraction per model.  Block (j, k) sums slice j of the invocations for model k in a fixed order; the
// block that finishes last for a model (a ticket counter, which it leaves at zero) adds the slices' partial sums in index
// order.  The result depends on neither the order nor the timing of the blocks.
__global__ void k_value_class(ValueArgs a) {
    __shared__ float sh[32];
    __shared__ int last;
    const int k = blockIdx.y, j = blockIdx.x, n_slices = gridDim.x;
    const int per = (a.n_inv + n_slices - 1) / n_slices;
    const int s_end = min(a.n_inv, (j + 1) * per);
    float sum = 0.f, clp = 0.f;
#pragma unroll 4
    for (int s = j * per + threadIdx.x; s < s_end; s += 1024) {
        const int role = a.inv_role[s];
        const float l = a.inv_sums[s * 3 + 1], c = a.inv_sums[s * 3 + 2];
        const bool mine = role >= 0 && role < a.n_roles && a.role_model[role] == k;
        sum += mine ? l : 0.f;
        clp += mine ? c : 0.f;
    }
    sum = block_sum_1024(sum, sh);
    clp = block_sum_1024(clp, sh);
    if (threadIdx.x == 0) {
        a.partial[(k * kValueSlices + j) * 2 + 0] = sum;
        a.partial[(k * kValueSlices + j) * 2 + 1] = clp;
        __threadfence();
        last = atomicAdd(&a.tickets[k], 1) == n_slices - 1;
    }
    __syncthreads();
    if (!last || threadIdx.x != 0) return;
    __threadfence();
    float tot = 0.f, tot_c = 0.f;
    for (int q = 0; q < n_slices; ++q) {
        tot += __ldcg(&a.partial[(k * kValueSlices + q) * 2 + 0]);
        tot_c += __ldcg(&a.partial[(k * kValueSlices + q) * 2 + 1]);
    }
    a.tickets[k] = 0;
    a.loss[k] = tot / value_Mk(a, k);
    if (a.clip_frac) a.clip_frac[k] = tot_c / fmaxf(static_cast<float>(a.model_cnt[k]), 1.f);
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------------
size_t value_counters_bytes() { return sizeof(unsigned long long) * UNITY_MAX_MODELS + sizeof(int) * UNITY_MAX_MODELS; }

size_t advantage_table_bytes(long long n_seg) { return kSegHeaderBytes + static_cast<size_t>(n_seg) * 32; }

cudaError_t launch_advantage(const AdvArgs& a, cudaStream_t stream, int* n_launches) {
    const int n_seg = a.n_groups * a.n_roles;
    if (a.n_inv > 0 || a.seg_mean || a.seg_std) {
        cudaError_t e = cudaMemsetAsync(a.seg_table, 0, advantage_table_bytes(n_seg), stream);
        if (e != cudaSuccess) return e;
        const int n_fin = a.n_inv > n_seg ? a.n_inv : n_seg;
        const int want = (n_fin + 255) / 256;
        // blocks of k_adv_stats that fit the current device at once (0: no cooperative launch), looked up once per device
        static int resident_cache[64];
        static bool resident_known[64];
        int dev = 0;
        if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
        int resident = 0;
        if (dev >= 0 && dev < 64 && resident_known[dev]) {
            resident = resident_cache[dev];
        } else {
            int coop = 0, sms = 0, per_sm = 0;
            cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            if (coop && cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_adv_stats, 256, 0) == cudaSuccess)
                resident = sms * per_sm;
            cudaGetLastError();
            if (dev >= 0 && dev < 64) { resident_cache[dev] = resident; resident_known[dev] = true; }
        }
        if (resident > 0) {
            // one cooperative launch: every block resident, so the grid barriers between the passes cannot starve
            int phase = 0;
            AdvArgs args = a;
            void* params[2] = {&args, &phase};
            e = cudaLaunchCooperativeKernel(reinterpret_cast<void*>(k_adv_stats), dim3(want < resident ? want : resident), dim3(256),
                                            params, 0, stream);
            if (e != cudaSuccess) return e;
            *n_launches += 1;
        } else {
            cudaGetLastError();
            for (int phase = 1; phase <= 3; ++phase) k_adv_stats<<<want, 256, 0, stream>>>(a, phase);
            *n_launches += 3;
        }
    }
    const bool aligned = (reinterpret_cast<uintptr_t>(a.tok_mask) & 15) == 0 && (reinterpret_cast<uintptr_t>(a.adv_tok) & 15) == 0;
    if (a.n_tok > 0 && aligned && a.n_tok / a.n_inv >= 128 && a.n_inv >= 1024) {
        // long invocations, and enough of them to fill the machine: one warp each
        k_adv_broadcast_inv<<<(a.n_inv + 7) / 8, 256, 0, stream>>>(a);
        *n_launches += 1;
    } else if (a.n_tok > 0) {
        // enough blocks to fill the machine (about 8 per SM), at most 32 rounds per block
        long long rounds = a.n_tok / (1024LL * 148 * 8);
        rounds = rounds < 1 ? 1 : (rounds > 32 ? 32 : rounds);
        const long long per_block = 1024 * rounds;
        k_adv_broadcast<<<static_cast<unsigned>((a.n_tok + per_block - 1) / per_block), 256, 0, stream>>>(
            a, static_cast<int>(rounds));
        *n_launches += 1;
    }
    return cudaGetLastError();
}

cudaError_t launch_route(const RouteArgs& a, cudaStream_t stream, int* n_launches) {
    k_route_count<<<a.n_blocks, kRouteBlock, 0, stream>>>(a);
    k_route_scan<<<1, 1024, 0, stream>>>(a);
    k_route_assign<<<a.n_blocks, kRouteBlock, 0, stream>>>(a);
    *n_launches += 3;
    return cudaGetLastError();
}

cudaError_t launch_gather_rows(const __nv_bfloat16* hidden, const int32_t* target, const int* slot_tok,
                               const DevPlan* plan, int K, long long max_slots, int H, __nv_bfloat16* hp, int* target_p,
                               cudaStream_t stream) {
    if (max_slots == 0) return cudaSuccess;
    k_gather_rows<<<static_cast<unsigned>((max_slots + 7) / 8), 256, 0, stream>>>(hidden, target, slot_tok, plan, K, H, hp,
                                                                                  target_p);
    return cudaGetLastError();
}

cudaError_t launch_finish_rows(const TokenArgs& a, bool with_loss, cudaStream_t stream, int* n_launches) {
    const long long n = a.block.model >= 0 ? a.block.row_cap : a.max_slots;      // bound of the rows; the kernel knows the extent
    if (n > 0) {
        k_finish_rows<<<(n + 255) / 256, 256, 0, stream>>>(a, with_loss ? 1 : 0);
        *n_launches += 1;
    }
    return cudaGetLastError();
}

cudaError_t launch_loss_reduce(const TokenArgs& a, cudaStream_t stream, int* n_launches) {
    if (a.n_inv > 0) {
        k_inv_reduce<<<(a.n_inv + 7) / 8, 256, 0, stream>>>(a);
        *n_launches += 1;
    }
    k_class_reduce<<<(a.K + a.n_roles + 7) / 8, 256, 0, stream>>>(a);
    *n_launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_finish_forward(const TokenArgs& a, bool with_loss, cudaStream_t stream, int* n_launches) {
    cudaError_t e = launch_finish_rows(a, with_loss, stream, n_launches);
    if (e != cudaSuccess || !with_loss) return e;
    return launch_loss_reduce(a, stream, n_launches);
}

cudaError_t launch_logit_grad_inplace(const LogitGradArgs& a, cudaStream_t stream) {
    if (a.span.row_cap <= 0 || a.cols <= 0) return cudaSuccess;
    // a block covers 8192 columns of one row; y walks the rows (grid-stride, the y extent is limited to 65535)
    const unsigned gx = static_cast<unsigned>((a.cols + 8191) / 8192);
    const unsigned gy = static_cast<unsigned>(a.span.row_cap < 32768 ? a.span.row_cap : 32768);
    k_logit_grad_inplace<<<dim3(gx, gy), 256, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_zero_masked_rows(const int* tok_slot, long long n_tok, int H, __nv_bfloat16* dHidden,
                                    cudaStream_t stream) {
    if (n_tok == 0) return cudaSuccess;
    k_zero_masked_rows<<<static_cast<unsigned>((n_tok + 7) / 8), 256, 0, stream>>>(tok_slot, n_tok, H, dHidden);
    return cudaGetLastError();
}

cudaError_t launch_store_dhidden(const float* dHc, const int* slot_tok, const RowSpan& span, int H,
                                 __nv_bfloat16* dHidden, cudaStream_t stream) {
    if (span.row_cap == 0) return cudaSuccess;
    k_store_dhidden<<<(span.row_cap + 7) / 8, 256, 0, stream>>>(dHc, slot_tok, span, H, dHidden);
    return cudaGetLastError();
}

cudaError_t launch_zero_if_empty(float* dst, long long n, const DevPlan* plan, int k, cudaStream_t stream) {
    if (n == 0) return cudaSuccess;
    k_zero_if_empty<<<1184, 256, 0, stream>>>(reinterpret_cast<float4*>(dst), n >> 2, plan, k);
    return cudaGetLastError();
}

cudaError_t launch_gae(int n_inv, const int64_t* cu_seqlens, const float* rewards, const float* values,
                       const uint8_t* tok_mask, float gamma, float lam, float* adv, float* ret, cudaStream_t stream) {
    if (n_inv == 0) return cudaSuccess;
    GaeArgs a{n_inv, cu_seqlens, rewards, values, tok_mask, gamma, lam, adv, ret};
    const uintptr_t al = reinterpret_cast<uintptr_t>(rewards) | reinterpret_cast<uintptr_t>(values) |
                         reinterpret_cast<uintptr_t>(adv) | reinterpret_cast<uintptr_t>(ret);
    if ((al & 15) == 0 && (reinterpret_cast<uintptr_t>(tok_mask) & 3) == 0)
        k_gae_vec<<<(n_inv + 7) / 8, 256, 0, stream>>>(a);
    else
        k_gae<<<(n_inv + 7) / 8, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_reward_assembly(const RewardArgs& a, cudaStream_t stream) {
    if (a.n_inv == 0) return cudaSuccess;
    k_reward_assembly<<<(a.n_inv + 255) / 256, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_value_loss(const ValueArgs& a, cudaStream_t stream, int* n_launches) {
    const int gi = (a.n_inv + 7) / 8;
    // per-model token counts and the tickets of the last pass start at zero (one small clear)
    cudaError_t e = cudaMemsetAsync(a.model_cnt, 0, value_counters_bytes(), stream);
    if (e != cudaSuccess) return e;
    if (a.n_inv > 0) { k_value_count<<<gi, 256, 0, stream>>>(a); *n_launches += 1; }
    if (a.n_inv > 0) { k_value_main<<<gi, 256, 0, stream>>>(a); *n_launches += 1; }
    int slices = (a.n_inv + 2047) / 2048;
    slices = slices < 1 ? 1 : (slices > kValueSlices ? kValueSlices : slices);
    k_value_class<<<dim3(slices, a.K), 1024, 0, stream>>>(a);
    *n_launches += 1;
    return cudaGetLastError();
}

}  // namespace unity
