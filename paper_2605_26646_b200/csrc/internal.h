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
// GEMM  C[m, n] = sum_k A[m, k] * B[n, k]   (bf16 operands, K-major or MN-major, fp32 accumulation in TMEM)
// ----------------------------------------------------------------------------------------------
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
    // ... and the last round, when it holds fewer row tiles than the others, may cut the vocabulary into more splits so
    // that it still occupies the machine: row tiles >= last_m0 use last_splits / last_tiles_per_split and write their
    // statistics to stats[last_stats_off + split * last_pitch + (row - first row of tile last_m0)]
    int last_m0, last_splits, last_tiles_per_split;
    long long last_stats_off, last_pitch;
    unsigned* round_counter;  // ever-growing arrival counter (null = no rendezvous between rounds)
    unsigned round_base;      // its value before this launch
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
cudaError_t launch_gemm(GemmEpilogue epi, bool a_mn, int ctas, const CUtensorMap& tmA, const CUtensorMap& tmB,
                        const GemmArgs& args, int sm_count, cudaStream_t stream, bool wide = false);
// Arrivals the launch adds to args.round_counter (rounds x workers); 0 when nothing is launched.
unsigned gemm_round_arrivals(GemmEpilogue epi, int ctas, const GemmArgs& args, int sm_count);
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
    int* counts;                 // [K] valid rows per model
    int* offsets;                // [K+1] first slot of each model (multiples of kTileM), offsets[K] = total slots
    int* tok_slot;               // [n_tok] slot of a token or -1
    int* slot_tok;               // [max_slots] token of a slot or -1 (pre-filled with -1)
    int8_t* tok_model;           // [n_tok] model id or -1
    int* status;
};
cudaError_t launch_route(const RouteArgs& a, cudaStream_t stream, int* n_launches);

cudaError_t launch_gather_rows(const __nv_bfloat16* hidden, const int32_t* target, const int* slot_tok, int n_slots,
                               int H, __nv_bfloat16* hp, int* target_p, cudaStream_t stream);

struct TokenArgs {
    int slot_begin;            // k_finish_rows works on slots [slot_begin, n_slots)
    int n_slots, n_splits, K, n_roles, n_inv;
    long long n_tok;
    const float4* stats;       // per model: base stats_base[k], pitch = padded rows of the model
    long long stats_base[UNITY_MAX_MODELS];
    int model_splits[UNITY_MAX_MODELS];
    // rows of a model from last_row0[k] on (relative to its first slot) were swept with last_splits[k] splits; their
    // statistics start at stats_last[k] with pitch = the model's padded rows - last_row0[k]
    int last_row0[UNITY_MAX_MODELS];
    int last_splits[UNITY_MAX_MODELS];
    long long stats_last[UNITY_MAX_MODELS];
    const int* slot_tok;
    const int* tok_slot;
    const int8_t* tok_model;
    int offsets[UNITY_MAX_MODELS + 1];
    float scale;               // inv_temperature
    // forward outputs (packed and caller order)
    float *row_lse, *row_ent, *row_logp;      // packed [n_slots]
    float *logp, *entropy, *lse;              // caller order [n_tok], nullable
    const float *logp_in, *entropy_in, *lse_in;   // caller order [n_tok]: results of an earlier forward (or all null)
    // loss part (null for logprob_fwd)
    const float *old_logp, *ref_logp, *adv_tok;
    float clip_lo, clip_hi, kl_coef, ent_coef;
    int kl_mode;
    float norm[UNITY_MAX_MODELS];   // M_k
    float *coef_a, *coef_b;    // packed [n_slots], already multiplied by scale
    float* tok_loss;           // caller order, nullable
    const int64_t* cu_seqlens;
    const int32_t* inv_role;
    int32_t role_model[UNITY_MAX_ROLES];
    float* inv_sums;           // [n_inv * 9]
    float* loss;               // [K]
    float* metrics;            // [(K + n_roles) * 8] nullable
};
cudaError_t launch_finish_forward(const TokenArgs& a, bool with_loss, cudaStream_t stream, int* n_launches);
// the two halves of the above: per-row terms for slots [a.slot_begin, a.n_slots), and the loss / metric reductions
cudaError_t launch_finish_rows(const TokenArgs& a, bool with_loss, cudaStream_t stream, int* n_launches);
cudaError_t launch_loss_reduce(const TokenArgs& a, cudaStream_t stream, int* n_launches);

// In place, for a block of rows x cols (row pitch ld) of stashed scaled logits z: z <- dL/dz =
// -p*(a + b*(z - lse + H)) (+ a at the target), p = exp(z - lse); per-row vectors are indexed from `row0`.
struct LogitGradArgs {
    __nv_bfloat16* Z;
    long long ld;
    int rows, cols, row0, vocab0;
    const int* target_p;
    const float *coef_a, *coef_b, *row_lse, *row_ent;
};
cudaError_t launch_logit_grad_inplace(const LogitGradArgs& a, cudaStream_t stream);

cudaError_t launch_zero_masked_rows(const int* tok_slot, long long n_tok, int H, __nv_bfloat16* dHidden,
                                    cudaStream_t stream);
// dHidden[slot_tok[slot0 + r], :] = bf16(dHc[r, :]) for r < n_rows with a token
cudaError_t launch_store_dhidden(const float* dHc, const int* slot_tok, int slot0, int n_rows, int H,
                                 __nv_bfloat16* dHidden, cudaStream_t stream);

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
    float* Mk;          // [2 * UNITY_MAX_MODELS] denominators M_k, then max(valid tokens, 1) per model
    float *loss, *clip_frac, *tok_loss, *dvalues;
    int* status;
};
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
