// Internal declarations shared by the translation units of libunity (not part of the C ABI).
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/unity.h"

namespace unity {

constexpr int kTileM = 256;   // rows of one output tile, shared by a pair of CTAs; row groups are padded to this
constexpr int kCtaM = 128;    // rows of A per CTA of the pair (= TMEM lanes)
constexpr int kTileN = 256;   // columns of one output tile (TMEM columns per accumulator stage)
constexpr int kBoxRows = 128; // rows of a K-major TMA box (A and B alike)
constexpr int kTileK = 64;    // bf16 elements per shared-memory K slab (one 128-byte swizzle row)
constexpr int kRouteBlock = 256;          // threads (= tokens) per block in the routing kernels
constexpr long long kWaitBudgetCycles = 4000000000LL;   // ~2 s: default bound of every in-kernel wait (GemmArgs::wait_budget)

// Device status bits (sticky, ORed into the context's status word).
constexpr int kStatusBadIndex = 1;
constexpr int kStatusTimeout = 2;

// ----------------------------------------------------------------------------------------------
// Row layout on the device.  The number of valid rows per model is known only after the routing kernels have run, and
// the host never reads it back (the calls stay asynchronous): every kernel whose extent depends on it takes the plan
// and a span of rows and works out its own extent; a launch whose span turns out empty returns at once.
// ----------------------------------------------------------------------------------------------
struct DevPlan {
    int counts[UNITY_MAX_MODELS];             // valid rows per model
    int off[UNITY_MAX_MODELS + 1];            // first packed slot per model (multiples of kTileM); off[K] = slots in use
    long long stats_base[UNITY_MAX_MODELS];   // first float4 of model k's forward statistics
};
// Rows [row_begin, row_begin + row_cap) of `model`'s packed range, cut to the rows the model has.
struct RowSpan {
    const DevPlan* plan;
    int model, row_begin, row_cap;
};
__device__ __forceinline__ void span_resolve(const RowSpan& s, int& slot0, int& n_rows) {
    const int first = s.plan->off[s.model];
    const int rows = s.plan->off[s.model + 1] - first;
    const int left = rows - s.row_begin;
    n_rows = left < 0 ? 0 : (left < s.row_cap ? left : s.row_cap);
    slot0 = first + s.row_begin;
}

// Shape of one forward launch over `rows` packed rows (a multiple of the row tile): row tiles per round and
// vocabulary splits.  One round of the persistent kernel = gm row tiles x splits vocabulary splits <= number of
// workers (CTAs or CTA pairs): gm bounds the hidden rows that must stay L2 resident (48 tiles of 128 rows by default:
// 6 k rows, 44 MB at H = 3584, loaded with an evict-last hint), splits fill the machine.  Computed identically
// wherever it is needed (the forward kernel, the kernel that merges its splits, the host's size bounds).
struct FwdShape {
    int gm, splits, tps;                  // row tiles per round; vocabulary splits and tiles per split of a full round
    int last_m0, last_splits, last_tps;   // first row tile, splits and tiles per split of a short last round
                                          // (last_m0 = number of row tiles when the last round is like the others)
    long long stats_rows;                 // float4 entries the launch writes: splits x rows + last_splits x last rows
};
struct FwdPlanParams {
    int n_pairs;     // workers (CTAs or CTA pairs) of the forward kernel
    int gmax;        // largest round, in row tiles
    int tile_rows;   // rows of a row tile (128 or 256)
    int n_tiles;     // vocabulary tiles of 256
};
__host__ __device__ inline FwdShape forward_shape(const FwdPlanParams& p, int rows) {
    const int m_tiles = rows / p.tile_rows;
    // Among round sizes from two thirds of gmax up to gmax, take the one with the least work per worker: vocabulary
    // tiles per split, summed over the rounds, the last of which may hold fewer row tiles and then cuts the vocabulary
    // into more splits (a batch whose row tiles do not divide well would otherwise idle part of the machine in its
    // last round); ties go to the larger round, which streams W less often.
    FwdShape best;
    best.gm = 1; best.splits = 1; best.tps = p.n_tiles; best.last_m0 = m_tiles; best.last_splits = 1; best.last_tps = p.n_tiles;
    long long best_cost = -1;
    const int cand_min = m_tiles <= p.gmax ? 1 : (2 * p.gmax + 2) / 3;      // few row tiles: any round size is L2-safe
    for (int cand = p.gmax; cand >= cand_min; --cand) {
        const int c = cand < m_tiles ? cand : (m_tiles > 0 ? m_tiles : 1);
        int sp = p.n_pairs / c;
        sp = sp > 32 ? 32 : sp;
        sp = sp > p.n_tiles ? p.n_tiles : sp;
        sp = sp < 1 ? 1 : sp;
        // several rounds: at most 4 splits, which bounds the statistics a launch writes by 4 per row (plus the short last
        // round's, at most one per worker and tile row); only a round size far below the default runs into this
        if (c < m_tiles && sp > 4) sp = 4;
        const int full_rounds = m_tiles / c, rest = m_tiles - full_rounds * c;
        int sp_last = sp;
        if (rest > 0) {
            sp_last = p.n_pairs / rest;
            sp_last = sp_last > 32 ? 32 : sp_last;
            sp_last = sp_last > p.n_tiles ? p.n_tiles : sp_last;
            sp_last = sp_last < 1 ? 1 : sp_last;
        }
        const long long cost = static_cast<long long>(full_rounds) * ((p.n_tiles + sp - 1) / sp) +
                               (rest > 0 ? (p.n_tiles + sp_last - 1) / sp_last : 0);
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            best.gm = c;
            best.tps = (p.n_tiles + sp - 1) / sp;
            best.splits = (p.n_tiles + best.tps - 1) / best.tps;
            best.last_m0 = rest > 0 && sp_last != sp ? full_rounds * c : m_tiles;
            best.last_tps = (p.n_tiles + sp_last - 1) / sp_last;
            best.last_splits = (p.n_tiles + best.last_tps - 1) / best.last_tps;
        }
    }
    const long long last_rows = static_cast<long long>(m_tiles - best.last_m0) * p.tile_rows;
    best.stats_rows = static_cast<long long>(best.splits) * rows + best.last_splits * last_rows;
    return best;
}

// ----------------------------------------------------------------------------------------------
// GEMM  C[m, n] = sum_k A[m, k] * B[n, k]   (bf16 operands, K-major or MN-major, fp32 accumulation in TMEM)
// ----------------------------------------------------------------------------------------------
enum : int { kSpanNone = 0, kSpanForward = 1, kSpanRowsA = 2, kSpanRowsM = 3, kSpanRowsK = 4 };
enum GemmEpilogue : int {
    kEpiSoftmaxStats = 0,   // online (max, sum exp, sum exp*z, target logit) per row; nothing of size M x N stored
    kEpiLogitGrad = 1,      // dL/dz in bf16 for a bounded (rows x vocab) chunk
    kEpiAccumF32 = 2        // C (+)= acc, fp32, row-major
};

struct GemmArgs {
    // tile grid and coordinates into the tensor maps
    int m_tiles, n_tiles, k_iters;   // tiles are gemm_tile_rows(ctas) x kTileN
    int group_m;              // row tiles per raster group (consecutive units share these A tiles)
    int a_row0, b_row0;       // first row of A / B (tensor-map coordinates) of tile (0, 0)
    int a_k0, b_k0;           // first K element of A / B
    int m_rows, n_cols;       // valid extent of C from (a_row0, b_row0): epilogue writes nothing beyond it
    // kEpiSoftmaxStats: a unit is (row tile, vocabulary split); a CTA keeps a unit's running statistics
    int n_splits, tiles_per_split;
    int n_active;             // workers that ever hold a unit (0 = all launched): the others leave at once and the round
                              // rendezvous counts only these
    // ... and the last round, when it holds fewer row tiles than the others, may cut the vocabulary into more splits so
    // that it still occupies the machine: row tiles >= last_m0 use last_splits / last_tiles_per_split and write their
    // statistics to stats[last_stats_off + split * last_pitch + (row - first row of tile last_m0)]
    int last_m0, last_splits, last_tiles_per_split;
    long long last_stats_off, last_pitch;
    unsigned* round_counter;  // this launch's arrival counter, zero before the launch (null = no rendezvous between rounds)
    int unit_tiles;           // logit gradient outside rounds: column tiles per unit (0 or 1: one output tile per unit)
    int plan_runs;            // logit gradient, rows known on the device only: the kernel picks unit_tiles and group_m itself
                              // from fwd.n_pairs (workers) and fwd.gmax (row tiles in flight that fit L2)
    int sync_period;          // epilogues other than softmax: rendezvous at every sync_period-th tile of a worker (>= 1)
    float4* stats;            // [n_splits][stats_pitch], row relative to a_row0: (max acc, sum e, sum e*acc, target acc)
    long long stats_pitch;
    const int* target_p;      // [rows] packed targets (global vocabulary index), indexed from a_row0 + row
    int vocab0;               // global vocabulary index of B row b_row0
    float scale;              // inv_temperature (softmax) / unused otherwise
    __nv_bfloat16* Z;         // optional stash of the scaled logits (null = none): chunk zc holds columns
    long long ldz;            //   [zc * z_chunk_cols, ...) of every row, row pitch ldz, chunks z_chunk_stride apart;
    long long z_chunk_stride; //   the last of the z_chunks chunks also takes the columns beyond it
    int z_chunk_cols, z_chunks;
    // kEpiLogitGrad
    const float* coef_a;      // [rows] dL/dlogp * scale, packed order
    const float* coef_b;      // [rows] dL/dentropy * scale
    int has_ent;              // 0: every coef_b of the launch is zero (no entropy term): shorter epilogue
    const float* row_lse;     // [rows]
    const float* row_ent;     // [rows]
    __nv_bfloat16* G;         // [m_rows, ldg] chunk-local
    long long ldg;
    int g_wide_store;         // G and ldg allow 32-byte aligned row segments: 256-bit stores
    // kEpiAccumF32
    float* C;
    long long ldc;
    int beta;                 // 0: overwrite, 1: add to C
    int mma_n;                // columns per MMA block, a multiple of 32 up to 256 (a tile is 1 or 2 blocks wide); 256
                              // unless the output's width divides better (896 columns = 4 blocks of 224)
    int l2_hints;             // L2 eviction policy (0 normal, 1 first, 2 last): bits 0-1 A loads, 2-3 B loads, 4-5 G stores
    int* status;
    // Rows known on the device only (span.plan != null): the kernel derives the row extent of the launch from the plan
    //   kSpanForward : A rows = the span; m_tiles, the round / split shape (forward_shape) and, with stats_from_plan,
    //                  the base of the statistics follow from it
    //   kSpanRowsA   : A rows = the span inside the hidden rows (recompute): a_row0 += first slot, m_rows, m_tiles
    //   kSpanRowsM   : M extent = the span's length (dHidden: A is the chunk-local G): m_rows, m_tiles
    //   kSpanRowsK   : K extent = the span's length (dW): k_iters, b_k0 += first slot
    RowSpan span;
    int span_mode;
    int stats_from_plan;
    FwdPlanParams fwd;
    long long wait_budget;    // SM clocks after which an mbarrier wait gives up (kStatusTimeout)
    int test_drop_slab;       // test hook: the TMA producer of every worker leaves out one K slab of its first tile
                              // (neither the expected-bytes arrival nor the loads), so the waits behind it run out
};

// a_mn: A is MN-major (only for kEpiAccumF32, whose B operand is always MN-major).  For an MN-major operand
// a_row0 / b_row0 index the contiguous dimension of its tensor map and a_k0 / b_k0 its rows.
// ctas: 1 = one CTA per 128 x 256 tile, 2 = a CTA pair per 256 x 256 tile; args.m_tiles counts tiles of
// gemm_tile_rows(ctas) rows.
// wide: output tiles two MMA blocks wide (kEpiAccumF32 with ctas = 2 only); args.n_tiles then counts tiles of
// 2 * args.mma_n columns instead of args.mma_n.
// workers: CTAs (or CTA pairs) to launch when the caller knows how many units a round holds; 0 = the whole machine
// (a worker without a unit leaves at once).
cudaError_t launch_gemm(GemmEpilogue epi, bool a_mn, int ctas, const CUtensorMap& tmA, const CUtensorMap& tmB,
                        const GemmArgs& args, int sm_count, cudaStream_t stream, bool wide = false, int workers = 0);
int gemm_tile_rows(int ctas);
int gemm_mma_n(int n_cols);   // block width for an fp32-accumulate GEMM with n_cols output columns
cudaError_t gemm_set_attributes();

// ----------------------------------------------------------------------------------------------
// streaming kernels (advantage, routing, token terms); each returns the launch error
// ----------------------------------------------------------------------------------------------
struct AdvArgs {
    int n_inv, n_traj, n_roles, n_groups;
    const int32_t *inv_role, *inv_group, *inv_traj;
    const float *r_node, *r_turn, *r_traj;
    int has_lam;
    float lam[UNITY_MAX_ROLES * 3];
    float eps;
    int ddof;
    long long n_tok;
    const int64_t* cu_seqlens;
    const uint8_t* tok_mask;
    float *adv_inv, *adv_tok, *seg_mean, *seg_std;
    float* r_scratch;   // [n_inv] combined reward
    int* seg_scratch;   // [n_inv] segment id g * n_roles + v, or -1 for an invocation with an id out of range
    void* seg_table;    // advantage_table_bytes(n_groups * n_roles) bytes, 8-byte aligned; cleared by launch_advantage
    int* status;
};
cudaError_t launch_advantage(const AdvArgs& a, cudaStream_t stream, int* n_launches);
size_t advantage_table_bytes(long long n_seg);   // per-segment accumulators of the statistics passes

struct RouteArgs {
    long long n_tok;
    int n_inv, n_roles, K, V;
    const int64_t* cu_seqlens;
    const int32_t* inv_role;
    int32_t role_model[UNITY_MAX_ROLES];
    const int32_t* target;
    const uint8_t* tok_mask;
    int n_blocks;                // ceil(n_tok / kRouteBlock)
    int* blk_cnt;                // [n_blocks * K] -> exclusive prefix per model after the scan
    DevPlan* plan;               // out: valid rows, first slot (multiples of kTileM) and statistics base of each model
    FwdPlanParams fwd;           // inputs of the forward planner (for the statistics bases)
    int* tok_slot;               // [n_tok] slot of a token or -1
    int* slot_tok;               // [max_slots] token of a slot or -1 (pre-filled with -1)
    int8_t* tok_model;           // [n_tok] model id or -1
    int* status;
};
cudaError_t launch_route(const RouteArgs& a, cudaStream_t stream, int* n_launches);

// packs the rows of slots [0, plan->off[K]); max_slots bounds the grid
cudaError_t launch_gather_rows(const __nv_bfloat16* hidden, const int32_t* target, const int* slot_tok,
                               const DevPlan* plan, int K, long long max_slots, int H, __nv_bfloat16* hp, int* target_p,
                               cudaStream_t stream);

struct TokenArgs {
    // k_finish_rows works on the rows of `block` (block.model >= 0: one block of one model's rows, whose forward ran as
    // a launch of its own with its statistics at stats[0..]), or on every packed row (block.model < 0)
    RowSpan block;
    const DevPlan* plan;
    FwdPlanParams fwd;         // the forward planner's inputs: the split layout of the statistics follows from the rows
    long long max_slots;       // bound of the packed rows (sizes the grid)
    int K, n_roles, n_inv;
    long long n_tok;
    const float4* stats;       // per model: base plan->stats_base[k], pitch = padded rows of the model
    const int* slot_tok;
    const int* tok_slot;
    const int8_t* tok_model;
    float scale;               // inv_temperature
    // forward outputs (packed and caller order)
    float *row_lse, *row_ent, *row_logp;      // packed [slots]
    float *logp, *entropy, *lse;              // caller order [n_tok], nullable
    const float *logp_in, *entropy_in, *lse_in;   // caller order [n_tok]: results of an earlier forward (or all null)
    // loss part (null for logprob_fwd)
    const float *old_logp, *ref_logp, *adv_tok;
    float clip_lo, clip_hi, kl_coef, ent_coef;
    int kl_mode;
    int has_norm;                   // 1: M_k = norm[k]; 0: M_k = max(valid rows of model k, 1) from the plan
    float norm[UNITY_MAX_MODELS];
    float *coef_a, *coef_b;    // packed [slots], already multiplied by scale
    float* tok_loss;           // caller order, nullable
    const int64_t* cu_seqlens;
    const int32_t* inv_role;
    int32_t role_model[UNITY_MAX_ROLES];
    float* inv_sums;           // [n_inv * 9]
    float* loss;               // [K]
    float* metrics;            // [(K + n_roles) * 8] nullable
};
cudaError_t launch_finish_forward(const TokenArgs& a, bool with_loss, cudaStream_t stream, int* n_launches);
// the two halves of the above: per-row terms for the rows of a.block (or all packed rows), and the loss / metric reductions
cudaError_t launch_finish_rows(const TokenArgs& a, bool with_loss, cudaStream_t stream, int* n_launches);
cudaError_t launch_loss_reduce(const TokenArgs& a, cudaStream_t stream, int* n_launches);

// In place, for a block of rows x cols (row pitch ld) of stashed scaled logits z: z <- dL/dz =
// -p*(a + b*(z - lse + H)) (+ a at the target), p = exp(z - lse).
struct LogitGradArgs {
    __nv_bfloat16* Z;
    long long ld;
    RowSpan span;              // the rows of the block; per-row vectors are indexed from its first slot
    int cols, vocab0;
    const int* target_p;
    const float *coef_a, *coef_b, *row_lse, *row_ent;
};
cudaError_t launch_logit_grad_inplace(const LogitGradArgs& a, cudaStream_t stream);

cudaError_t launch_zero_masked_rows(const int* tok_slot, long long n_tok, int H, __nv_bfloat16* dHidden,
                                    cudaStream_t stream);
// dHidden[slot_tok[first slot of the span + r], :] = bf16(dHc[r, :]) for the rows r of the span that hold a token
cudaError_t launch_store_dhidden(const float* dHc, const int* slot_tok, const RowSpan& span, int H,
                                 __nv_bfloat16* dHidden, cudaStream_t stream);
// dst[0, n) = 0 when model k has no valid row (its dW when nothing accumulates into it)
cudaError_t launch_zero_if_empty(float* dst, long long n, const DevPlan* plan, int k, cudaStream_t stream);

cudaError_t launch_gae(int n_inv, const int64_t* cu_seqlens, const float* rewards, const float* values,
                       const uint8_t* tok_mask, float gamma, float lam, float* adv, float* ret, cudaStream_t stream);

struct RewardArgs {
    int n_inv, n_traj, n_roles, max_turns;
    const int32_t *inv_role, *inv_traj, *inv_turn;
    const float* score;          // [n_traj, max_turns]
    const int32_t* n_scores;     // [n_traj] or null (= max_turns)
    const uint8_t* inv_end;      // [n_inv] or null
    int mode[UNITY_MAX_ROLES];   // 0 none, 1 absolute, 2 marginal
    int shift[UNITY_MAX_ROLES];
    float* r_turn;               // out [n_inv]
    int* status;
};
cudaError_t launch_reward_assembly(const RewardArgs& a, cudaStream_t stream);

struct ValueArgs {
    int n_inv, n_roles, K;
    const int64_t* cu_seqlens;
    const int32_t* inv_role;
    int32_t role_model[UNITY_MAX_ROLES];
    const uint8_t* tok_mask;
    const float *values, *old_values, *returns;
    float clip_v;
    int has_norm;
    int vec_ok;         // token arrays 16-byte aligned and the mask 4-byte aligned: 128-bit accesses allowed
    float norm[UNITY_MAX_MODELS];
    float* inv_sums;    // [n_inv * 3] count, sum of token losses, clipped tokens
    unsigned long long* model_cnt;   // [UNITY_MAX_MODELS] valid tokens per model, directly followed by ...
    int* tickets;       // [UNITY_MAX_MODELS] ... the arrival counters of k_value_class (value_counters_bytes() in all)
    float* partial;     // [UNITY_MAX_MODELS * kValueSlices * 2] per-slice sums of k_value_class
    float *loss, *clip_frac, *tok_loss, *dvalues;
    int* status;
};
constexpr int kValueSlices = 32;      // slices of the invocations in the last pass of the value loss
size_t value_counters_bytes();
cudaError_t launch_value_loss(const ValueArgs& a, cudaStream_t stream, int* n_launches);

// ----------------------------------------------------------------------------------------------
// ready-batch construction (batch_kernels.cu)
// ----------------------------------------------------------------------------------------------
struct BatchArgs {
    int n_inv, n_traj, n_roles, K, n_parts, pad_to;
    int half_bits;               // half width of the Feistel domain
    uint32_t key[4];             // round keys derived from the seed
    const int64_t* cu_seqlens;
    const int32_t *inv_role, *inv_traj;
    const uint8_t* traj_done;
    int32_t role_model[UNITY_MAX_ROLES];   // -1: the role's tokens are not trained
    int n_blocks;                // ceil(n_inv / batch_block())
    // scratch
    int* pos_inv;                // [n_inv] invocation at each shuffled position
    int8_t* pos_model;           // [n_inv] its model, or -1 when dropped
    int* blk_cnt;                // [n_blocks * K] -> exclusive prefix per model
    long long* blk_tok;          // [n_blocks * K] same for padded tokens
    long long* model_tok;        // [K + 1] first padded token of each model
    // outputs
    int* order;                  // [n_inv]
    int64_t* out_cu;             // [n_inv + 1]
    int* model_offsets;          // [K + 1]
    int* part_offsets;           // [K * n_parts + 1]
    long long* totals;           // [2] kept invocations, padded tokens
    int* status;
};
void batch_keys(uint64_t seed, int n_inv, BatchArgs* a);
int batch_block();
cudaError_t launch_batch_plan(const BatchArgs& a, cudaStream_t stream, int* n_launches);

struct GatherArgs {
    int n_inv;                   // upper bound of kept invocations (sizes the grid)
    const int* order;
    const int64_t *src_cu, *out_cu;
    const long long* totals;
    long long row_bytes;         // bytes per token
    int unit_bytes;              // copy unit: 1, 2, 4, 8 or 16, dividing row_bytes and the alignment of src / dst
    long long avg_len;           // mean tokens per invocation (sizes the grid)
    const void* src;
    void* dst;
    unsigned char pad[16];       // pad pattern of pad_bytes bytes
    int pad_bytes;
};
cudaError_t launch_batch_gather(const GatherArgs& g, cudaStream_t stream);
cudaError_t launch_align_rewards(int n_inv, const int64_t* cu, const uint8_t* mask, const float* r_inv,
                                 float* tok_reward, cudaStream_t stream);

}  // namespace unity
