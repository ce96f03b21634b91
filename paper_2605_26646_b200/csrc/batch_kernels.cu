// Ready-batch construction on the device: the step between a model-local rollout buffer and the update calls.
//   plan   : seeded shuffle (a Feistel bijection of the position index, so no sort and no random-number state),
//            filter of invocations whose trajectory is incomplete or whose role is not trained, stable listing per
//            model, padded token offsets, and a token-balanced split of every model's list into contiguous partitions
//   gather : moves any token-level tensor of the buffer into the planned order (contiguous block copies + pad fill)
//   align  : puts a delayed, invocation-level reward on the last unmasked token of its sequence
// All integer work; every output is a pure function of the inputs (no atomics on results), so it is bit-exact.
#include <cstring>

#include "internal.h"

namespace unity {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kBatchBlock = 256;

// 32-bit finaliser of MurmurHash3.
__host__ __device__ __forceinline__ uint32_t fmix32(uint32_t h) {
    h ^= h >> 16; h *= 0x85ebca6bu; h ^= h >> 13; h *= 0xc2b2ae35u; h ^= h >> 16;
    return h;
}

// Position p of the shuffled order holds invocation feistel(p): four balanced Feistel rounds on the smallest
// even-width bit domain that holds n, re-applied while the value falls outside [0, n) (cycle walking: the map is a
// bijection of the domain, so the walk from p < n returns to [0, n) after finitely many steps).
__device__ __forceinline__ int shuffled_index(int p, int n, int half, const uint32_t* key) {
    const uint32_t hmask = (1u << half) - 1u;
    uint32_t x = static_cast<uint32_t>(p);
    do {
        uint32_t left = x >> half, right = x & hmask;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t f = fmix32(right ^ key[i]) & hmask;
            const uint32_t nl = right;
            right = left ^ f;
            left = nl;
        }
        x = (left << half) | right;
    } while (x >= static_cast<uint32_t>(n));
    return static_cast<int>(x);
}

__device__ __forceinline__ long long padded_len(const int64_t* cu, int s, int pad_to) {
    const long long len = cu[s + 1] - cu[s];
    return (len + pad_to - 1) / pad_to * pad_to;
}

// Pass 1: position -> invocation, keep / drop, model; per-block invocation and token counts per model.
__global__ void k_batch_count(BatchArgs a) {
    __shared__ int cnt[UNITY_MAX_MODELS];
    __shared__ unsigned long long tok[UNITY_MAX_MODELS];
    if (threadIdx.x < UNITY_MAX_MODELS) { cnt[threadIdx.x] = 0; tok[threadIdx.x] = 0ull; }
    __syncthreads();
    const int p = blockIdx.x * kBatchBlock + threadIdx.x;
    if (p < a.n_inv) {
        const int s = shuffled_index(p, a.n_inv, a.half_bits, a.key);
        int model = -1;
        const int role = a.inv_role[s], traj = a.inv_traj[s];
        if (role < 0 || role >= a.n_roles || traj < 0 || traj >= a.n_traj) {
            atomicOr(a.status, kStatusBadIndex);
        } else if (a.traj_done[traj] != 0) {
            model = a.role_model[role];                 // -1: a role that is not trained
        }
        a.pos_inv[p] = s;
        a.pos_model[p] = static_cast<int8_t>(model);
        if (model >= 0) {
            atomicAdd(&cnt[model], 1);                  // integer counts: order does not matter
            atomicAdd(&tok[model], static_cast<unsigned long long>(padded_len(a.cu_seqlens, s, a.pad_to)));
        }
    }
    __syncthreads();
    if (threadIdx.x < a.K) {
        a.blk_cnt[blockIdx.x * a.K + threadIdx.x] = cnt[threadIdx.x];
        a.blk_tok[blockIdx.x * a.K + threadIdx.x] = static_cast<long long>(tok[threadIdx.x]);
    }
}

// Pass 2 (one block): exclusive prefix over the blocks, per model, of both counts; model offsets and totals.
__global__ void k_batch_scan(BatchArgs a) {
    __shared__ long long part_c[1024];
    __shared__ long long part_t[1024];
    __shared__ long long total_c[UNITY_MAX_MODELS], total_t[UNITY_MAX_MODELS];
    const int tid = threadIdx.x, nt = blockDim.x;
    const int per = (a.n_blocks + nt - 1) / nt;
    const int b0 = min(tid * per, a.n_blocks), b1 = min(b0 + per, a.n_blocks);
    for (int k = 0; k < a.K; ++k) {
        long long sc = 0, st = 0;
        for (int b = b0; b < b1; ++b) { sc += a.blk_cnt[b * a.K + k]; st += a.blk_tok[b * a.K + k]; }
        part_c[tid] = sc; part_t[tid] = st;
        __syncthreads();
        for (int off = 1; off < nt; off <<= 1) {
            const long long vc = tid >= off ? part_c[tid - off] : 0, vt = tid >= off ? part_t[tid - off] : 0;
            __syncthreads();
            part_c[tid] += vc; part_t[tid] += vt;
            __syncthreads();
        }
        long long rc = part_c[tid] - sc, rt = part_t[tid] - st;
        if (tid == nt - 1) { total_c[k] = part_c[tid]; total_t[k] = part_t[tid]; }
        for (int b = b0; b < b1; ++b) {
            const int c = a.blk_cnt[b * a.K + k];
            const long long t = a.blk_tok[b * a.K + k];
            a.blk_cnt[b * a.K + k] = static_cast<int>(rc);
            a.blk_tok[b * a.K + k] = rt;
            rc += c; rt += t;
        }
        __syncthreads();
    }
    if (tid == 0) {
        long long oc = 0, ot = 0;
        for (int k = 0; k < a.K; ++k) {
            a.model_offsets[k] = static_cast<int>(oc);
            a.model_tok[k] = ot;
            oc += total_c[k]; ot += total_t[k];
        }
        a.model_offsets[a.K] = static_cast<int>(oc);
        a.model_tok[a.K] = ot;
        a.totals[0] = oc;
        a.totals[1] = ot;
    }
}

// Pass 3: every kept position finds its place: rank among the kept positions of its model before it (stable), and
// the padded tokens before it.
__global__ void k_batch_assign(BatchArgs a) {
    __shared__ int w_cnt[kBatchBlock / 32];
    __shared__ long long w_tok[kBatchBlock / 32];
    const int p = blockIdx.x * kBatchBlock + threadIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int model = p < a.n_inv ? a.pos_model[p] : -1;
    const int s = p < a.n_inv ? a.pos_inv[p] : 0;
    const long long len = model >= 0 ? padded_len(a.cu_seqlens, s, a.pad_to) : 0;
    int my_rank = 0;
    long long my_tok = 0;
    for (int k = 0; k < a.K; ++k) {
        const bool mine = model == k;
        const unsigned bal = __ballot_sync(kFull, mine);
        // inclusive warp scan of the token counts of this model's positions
        long long v = mine ? len : 0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const long long u = __shfl_up_sync(kFull, v, o);
            if (lane >= o) v += u;
        }
        if (lane == 31) { w_cnt[warp] = __popc(bal); w_tok[warp] = v; }
        __syncthreads();
        if (mine) {
            int rc = __popc(bal & ((1u << lane) - 1u));
            long long rt = v - len;
            for (int w = 0; w < warp; ++w) { rc += w_cnt[w]; rt += w_tok[w]; }
            my_rank = rc;
            my_tok = rt;
        }
        __syncthreads();
    }
    if (model < 0) return;
    const int j = a.model_offsets[model] + a.blk_cnt[blockIdx.x * a.K + model] + my_rank;
    a.order[j] = s;
    a.out_cu[j] = a.model_tok[model] + a.blk_tok[blockIdx.x * a.K + model] + my_tok;
}

// Pass 4: partition boundaries, and the tails of the outputs.  Invocation j of model k, with P_j padded tokens of the
// model before it, belongs to partition min(n_parts - 1, P_j * n_parts / T_k); partitions are contiguous, so the
// first member of each is found by comparing neighbours.
__device__ __forceinline__ int part_of(long long P, long long T, int n_parts) {
    if (T <= 0) return 0;
    const long long q = P * n_parts / T;
    return q < n_parts - 1 ? static_cast<int>(q) : n_parts - 1;
}

__global__ void k_batch_parts(BatchArgs a) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int n_kept = static_cast<int>(a.totals[0]);
    const long long n_tok = a.totals[1];
    if (j < a.K * a.n_parts) {                                   // models without a kept invocation
        const int k = j / a.n_parts;
        if (a.model_offsets[k + 1] == a.model_offsets[k]) a.part_offsets[j] = a.model_offsets[k];
    }
    if (j == 0) a.part_offsets[a.K * a.n_parts] = n_kept;
    if (j > a.n_inv) return;
    if (j >= n_kept) {
        a.out_cu[j] = n_tok;
        if (j < a.n_inv) a.order[j] = -1;
        return;
    }
    int k = 0;
    while (k + 1 < a.K && j >= a.model_offsets[k + 1]) ++k;
    const long long T = a.model_tok[k + 1] - a.model_tok[k];
    const int mine = part_of(a.out_cu[j] - a.model_tok[k], T, a.n_parts);
    const int prev = j == a.model_offsets[k] ? -1 : part_of(a.out_cu[j - 1] - a.model_tok[k], T, a.n_parts);
    for (int q = prev + 1; q <= mine; ++q) a.part_offsets[k * a.n_parts + q] = j;
    if (j == a.model_offsets[k + 1] - 1)
        for (int q = mine + 1; q < a.n_parts; ++q) a.part_offsets[k * a.n_parts + q] = j + 1;
}

// Gather: `slices` warps per kept invocation (one for per-token scalars, more for wide rows) copy the invocation's
// contiguous bytes and fill the pad; many invocations are in flight at once, so the chain order -> offsets -> data of
// one invocation overlaps with the copies of others.  When source and destination of an invocation are both 16-byte
// aligned, its whole 16-byte words move as 128-bit vectors whatever the unit T is (per-token scalars are contiguous
// across tokens); the rest, and unaligned invocations, move unit by unit.  Four accesses per lane are issued before
// their stores.
template <typename T>
__global__ void k_batch_gather(const int* __restrict__ order, const int64_t* __restrict__ src_cu,
                               const int64_t* __restrict__ out_cu, const long long* __restrict__ totals,
                               long long units_per_row, const T* __restrict__ src, T* __restrict__ dst, T pad, int slices) {
    const int n_kept = static_cast<int>(totals[0]);
    const long long warp = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int j = static_cast<int>(warp / slices);
    if (j >= n_kept) return;
    const long long stride = static_cast<long long>(slices) * 32;
    const long long first = (warp - static_cast<long long>(j) * slices) * 32 + (threadIdx.x & 31);
    const int s = order[j];
    const long long n_copy = (src_cu[s + 1] - src_cu[s]) * units_per_row;
    const long long n_slot = (out_cu[j + 1] - out_cu[j]) * units_per_row;
    const T* from = src + src_cu[s] * units_per_row;
    T* to = dst + out_cu[j] * units_per_row;
    long long done = 0;                                    // units already moved by the vector part
    if (sizeof(T) < 16 && ((reinterpret_cast<uintptr_t>(from) | reinterpret_cast<uintptr_t>(to)) & 15) == 0) {
        constexpr long long per = 16 / sizeof(T);
        const long long n_vec = n_copy / per;
        const uint4* from4 = reinterpret_cast<const uint4*>(from);
        uint4* to4 = reinterpret_cast<uint4*>(to);
        for (long long i = first; i < n_vec; i += 4 * stride) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const long long q = i + u * stride;
                if (q < n_vec) v[u] = from4[q];
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const long long q = i + u * stride;
                if (q < n_vec) to4[q] = v[u];
            }
        }
        done = n_vec * per;
    }
    for (long long i = done + first; i < n_slot; i += 4 * stride) {
        T v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long q = i + u * stride;
            v[u] = q < n_copy ? from[q] : pad;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long q = i + u * stride;
            if (q < n_slot) to[q] = v[u];
        }
    }
}

// Delayed rewards: one warp per invocation.  The sequence is zero-filled front to back; once the index is a multiple of
// 4 the warp covers 512 tokens per step (per lane four 32-bit mask loads and four 128-bit stores, each contiguous across
// the warp); every lane remembers the last unmasked token it saw, the warp takes the maximum, and after the warp's
// stores are ordered that token gets the reward.
__global__ void k_align_rewards(int n_inv, const int64_t* __restrict__ cu, const uint8_t* __restrict__ mask,
                                const float* __restrict__ r_inv, float* __restrict__ tok_reward, int vec_ok) {
    const int s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (s >= n_inv) return;
    const long long lo = cu[s], hi = cu[s + 1];
    long long last = -1;
    const long long head_end = vec_ok ? min(hi, (lo + 3) & ~3LL) : hi;
    for (long long t = lo + lane; t < head_end; t += 32) {
        tok_reward[t] = 0.f;
        if (mask == nullptr || mask[t]) last = t;
    }
    const long long n_quad = (hi - head_end) >> 2;
    for (long long q0 = 0; q0 < n_quad; q0 += 128) {
        unsigned m[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long q = q0 + u * 32 + lane;
            m[u] = 0u;
            if (q < n_quad) m[u] = mask == nullptr ? 0x01010101u : *reinterpret_cast<const unsigned*>(mask + head_end + (q << 2));
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long q = q0 + u * 32 + lane;
            if (q < n_quad) {
                const long long t = head_end + (q << 2);
                *reinterpret_cast<float4*>(tok_reward + t) = make_float4(0.f, 0.f, 0.f, 0.f);
                if (m[u]) last = t + ((31 - __clz(__vcmpne4(m[u], 0u))) >> 3);   // highest non-zero byte
            }
        }
    }
    for (long long t = head_end + (n_quad << 2) + lane; t < hi; t += 32) {
        tok_reward[t] = 0.f;
        if (mask == nullptr || mask[t]) last = t;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) last = max(last, __shfl_xor_sync(kFull, last, o));
    __syncwarp();                                   // the zero stores of all lanes are ordered before the reward's
    if (lane == 0 && last >= 0) tok_reward[last] = r_inv[s];
}

template <typename T>
cudaError_t gather_as(const GatherArgs& g, cudaStream_t stream) {
    T pad;
    // the pad pattern, replicated to the width of the copy unit
    unsigned char bytes[16];
    for (int i = 0; i < 16; ++i) bytes[i] = g.pad[i % g.pad_bytes];
    memcpy(&pad, bytes, sizeof(T));
    const long long units = g.row_bytes / static_cast<long long>(sizeof(T));
    // warps per invocation: one per 8 KiB of an average invocation, so that per-token scalars take one warp and rows
    // of hidden size spread over many
    long long slices = (g.row_bytes * g.avg_len + 8191) / 8192;
    slices = slices < 1 ? 1 : (slices > 1024 ? 1024 : slices);
    const long long warps = static_cast<long long>(g.n_inv > 0 ? g.n_inv : 1) * slices;
    k_batch_gather<T><<<static_cast<unsigned>((warps + 7) / 8), 256, 0, stream>>>(
        g.order, g.src_cu, g.out_cu, g.totals, units, static_cast<const T*>(g.src), static_cast<T*>(g.dst), pad,
        static_cast<int>(slices));
    return cudaGetLastError();
}

}  // namespace

void batch_keys(uint64_t seed, int n_inv, BatchArgs* a) {
    int bits = 2;
    while (bits < 31 && (1ll << bits) < n_inv) ++bits;
    bits += bits & 1;
    a->half_bits = bits / 2;
    const uint32_t seed32 = static_cast<uint32_t>(seed ^ (seed >> 32));
    for (int i = 0; i < 4; ++i) a->key[i] = fmix32(seed32 + 0x9E3779B9u * static_cast<uint32_t>(i + 1));
}

cudaError_t launch_batch_plan(const BatchArgs& a, cudaStream_t stream, int* n_launches) {
    if (a.n_inv > 0) {
        k_batch_count<<<a.n_blocks, kBatchBlock, 0, stream>>>(a);
        *n_launches += 1;
    }
    k_batch_scan<<<1, 1024, 0, stream>>>(a);
    if (a.n_inv > 0) {
        k_batch_assign<<<a.n_blocks, kBatchBlock, 0, stream>>>(a);
        *n_launches += 1;
    }
    const int n_threads = max(a.n_inv + 1, a.K * a.n_parts);
    k_batch_parts<<<(n_threads + 255) / 256, 256, 0, stream>>>(a);
    *n_launches += 2;
    return cudaGetLastError();
}

int batch_block() { return kBatchBlock; }

cudaError_t launch_batch_gather(const GatherArgs& g, cudaStream_t stream) {
    switch (g.unit_bytes) {
        case 16: return gather_as<uint4>(g, stream);
        case 8: return gather_as<uint2>(g, stream);
        case 4: return gather_as<uint32_t>(g, stream);
        case 2: return gather_as<uint16_t>(g, stream);
        default: return gather_as<uint8_t>(g, stream);
    }
}

cudaError_t launch_align_rewards(int n_inv, const int64_t* cu, const uint8_t* mask, const float* r_inv,
                                 float* tok_reward, cudaStream_t stream) {
    if (n_inv == 0) return cudaSuccess;
    const int vec_ok = (reinterpret_cast<uintptr_t>(mask) & 15) == 0 && (reinterpret_cast<uintptr_t>(tok_reward) & 15) == 0;
    k_align_rewards<<<(n_inv + 7) / 8, 256, 0, stream>>>(n_inv, cu, mask, r_inv, tok_reward, vec_ok);
    return cudaGetLastError();
}

}  // namespace unity
