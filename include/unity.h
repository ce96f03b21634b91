/*
 * unity.h - C ABI of libunity: the per-token policy computation of a multi-agent PPO update
 * (role-level advantages; grouped LM-head log-prob / entropy; PPO-clip + KL loss with backward)
 * for one NVIDIA B200 (sm_100a).
 *
 * Conventions
 * -----------
 * - Every function returns an int status: 0 (UNITY_OK) or a negative UNITY_ERR_* code.  Nothing
 *   throws, aborts or traps.  unity_last_error() gives a text for the last failure of a context.
 * - Unless marked (host), data pointers are DEVICE pointers owned by the caller; the library never
 *   frees or keeps them beyond the call.  Arrays marked (host) are read during the call.
 * - Work is enqueued on the stream given to unity_create and every call is asynchronous: the only
 *   calls that synchronise are unity_check_status, unity_get_profile and unity_destroy (and, when
 *   UNITY_OPT_HOST_COUNTS is set to 1, unity_logprob_fwd and unity_ppo_loss_fwd_bwd, once each, to
 *   read the K per-model row counts and skip launches that would be empty).  Device-side errors
 *   (bad indices in the data, a bounded wait that expired) are sticky in a status word read by
 *   unity_check_status.
 * - The library allocates no device memory per call: all scratch lives in the caller's workspace.
 * - Rows with tok_mask == 0 receive 0 in every per-token output and cost no tensor work.
 * - Limits: 1 <= K <= UNITY_MAX_MODELS, 1 <= n_roles <= UNITY_MAX_ROLES, H % 64 == 0, V % 8 == 0,
 *   hidden / W / dHidden / dW base addresses 16-byte aligned and densely packed (row pitch = H).
 * - One context per stream; a context is not re-entrant.
 */
#ifndef UNITY_H_
#define UNITY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define UNITY_OK 0
#define UNITY_ERR_INVALID_ARG (-1)   /* null pointer, negative size, parameter out of range      */
#define UNITY_ERR_SHAPE (-2)         /* H, V, K, n_roles outside the limits above                */
#define UNITY_ERR_ALIGNMENT (-3)     /* a matrix pointer is not 16-byte aligned                  */
#define UNITY_ERR_WORKSPACE (-4)     /* workspace smaller than unity_workspace_bytes(...)        */
#define UNITY_ERR_CUDA (-5)          /* a CUDA runtime / driver call failed                      */
#define UNITY_ERR_UNSUPPORTED_ARCH (-6) /* device is not compute capability 10.x                 */
#define UNITY_ERR_BAD_INDEX (-7)     /* device status: target / role / group / model id out of range;
                                        the offending row or invocation was treated as masked    */
#define UNITY_ERR_TIMEOUT (-8)       /* device status: a bounded in-kernel wait expired          */

#define UNITY_MAX_MODELS 16
#define UNITY_MAX_ROLES 64
#define UNITY_N_METRICS 8            /* per class: n_valid, mean pg loss, mean KL, mean entropy,
                                        clip fraction, mean ratio, mean logp, mean advantage     */

typedef struct unity_ctx unity_ctx;

/* Create a context bound to `device` and `cuda_stream` (a cudaStream_t; NULL = default stream).
 * `workspace` is caller-owned device memory of `workspace_bytes` bytes (256-byte aligned) that the
 * context uses as scratch until unity_destroy.  Fails with UNITY_ERR_UNSUPPORTED_ARCH off sm_100. */
int unity_create(unity_ctx** out, int device, void* cuda_stream, void* workspace, size_t workspace_bytes);
int unity_destroy(unity_ctx* ctx);

/* Scratch bytes sufficient for every call on batches of up to n_tok tokens of K models with these H and V,
 * whatever the number of invocations (it assumes n_inv <= n_tok and includes the bounded logit-gradient chunk).
 * Equal to unity_workspace_bytes(n_tok, H, V, K, n_tok); callers that know n_inv can ask for less below. */
size_t unity_workspace_hint(int64_t n_tok, int32_t H, int32_t V, int32_t K);
/* Scratch bytes that make every call with these sizes run with full-size chunks.  A smaller
 * workspace still works down to unity_workspace_min_bytes (smaller gradient chunks). */
size_t unity_workspace_bytes(int64_t n_tok, int32_t H, int32_t V, int32_t K, int32_t n_inv);
size_t unity_workspace_min_bytes(int64_t n_tok, int32_t H, int32_t V, int32_t K, int32_t n_inv);
/* Scratch bytes that leave room for the logit stash of UNITY_OPT_LOGIT_STASH. */
size_t unity_workspace_bytes_stash(int64_t n_tok, int32_t H, int32_t V, int32_t K, int32_t n_inv);

/* Synchronise the stream, return the sticky device status (UNITY_OK, UNITY_ERR_BAD_INDEX,
 * UNITY_ERR_TIMEOUT or UNITY_ERR_CUDA) and clear it. */
int unity_check_status(unity_ctx* ctx);
const char* unity_last_error(const unity_ctx* ctx);

/* Number of kernels this context has launched since creation (for benchmark bookkeeping). */
int64_t unity_launch_count(const unity_ctx* ctx);

/* Measurement hooks (no counterpart in the paper).  With profiling enabled, each tensor-core GEMM launch
 * of unity_ppo_loss_fwd_bwd / unity_logprob_fwd is bracketed by a CUDA event pair on
 * the context's stream.  unity_get_profile synchronises the stream, returns per class the summed device
 * time in milliseconds (ms[UNITY_PROF_CLASSES]) and the number of launches, and resets the counters. */
#define UNITY_PROF_FWD_GEMM 0   /* LM-head GEMM fused with online log-softmax / gather / entropy */
#define UNITY_PROF_GRAD_GEMM 1  /* logit recompute fused with dL/dz                              */
#define UNITY_PROF_DH_GEMM 2    /* dHidden chunk GEMM                                            */
#define UNITY_PROF_DW_GEMM 3    /* dW chunk GEMM                                                 */
#define UNITY_PROF_CLASSES 4
int unity_set_profiling(unity_ctx* ctx, int enable);

/* Tuning knobs (no counterpart in the paper).  Each GEMM class can run with one CTA per 128 x 256 output tile
 * (value 1) or with a pair of CTAs on neighbouring SMs sharing a 256 x 256 tile (value 2).  Results do not depend
 * on the choice beyond fp32 summation order inside the tensor core.  Defaults: 2, 2, 2, 2 (measured best on
 * the H=3584, V=152064 workload; all choices are within a few per cent under the 1 kW power cap). */
#define UNITY_OPT_CTAS_FWD 0
#define UNITY_OPT_CTAS_GRAD 1
#define UNITY_OPT_CTAS_DH 2
#define UNITY_OPT_CTAS_DW 3
#define UNITY_OPT_L2_PROMOTION 4  /* TMA tensor-map L2 promotion: 0 none, 1 64 B, 2 128 B, 3 256 B (default)          */
#define UNITY_OPT_CHUNK_GROUP 5   /* raster group of all three gradient-chunk GEMMs in 128-row tiles (defaults 40, 32, 32)       */
#define UNITY_OPT_CHUNK_ROWS 6    /* gradient chunk rows = value x 18944 (default 2; larger needs a larger workspace)   */
#define UNITY_OPT_CHUNK_VOCAB 7   /* gradient chunk vocabulary entries = value x 18944 (default 2)                      */
#define UNITY_OPT_FWD_GROUP 8     /* 128-row tiles per round of the forward kernel; 0 = a quarter of the SMs; -1 (default): half
                                     the SMs where that many hidden rows fit a 45 MB share of L2 (H <= 2368), else 48 */
#define UNITY_OPT_FWD_SYNC 9      /* 1 (default): workers of the forward kernel meet at each round start (bounded wait) */
#define UNITY_OPT_CHUNK_SYNC 10   /* same for the gradient-chunk GEMMs: bit 0 recompute, bit 1 dHidden, bit 2 dW (default 7) */
#define UNITY_OPT_WIDE_ACC 11     /* 1 (default): the dHidden / dW chunk GEMMs of CTA pairs use 256 x 512 output tiles    */
#define UNITY_OPT_GROUP_GRAD 12   /* raster group of the recompute GEMM alone, in 128-row tiles                           */
#define UNITY_OPT_GROUP_DH 13     /* ... of the dHidden GEMM                                                               */
#define UNITY_OPT_GROUP_DW 14     /* ... of the dW GEMM                                                                    */
#define UNITY_OPT_LOGIT_STASH 15  /* 0 (default): the backward recomputes the logits per vocabulary chunk.  1: the loss call
                                     runs its forward block by block of 18432 rows and keeps the block's scaled logits in
                                     bf16 (rows x V, about 6 GB at V = 152064, sized by unity_workspace_bytes_stash); the
                                     backward turns them into dL/dz in place.  Executed work drops from 8 to 6 H V flop per
                                     token; the full n_tok x V logits still never exist.  Ignored (recompute) when the
                                     workspace has no room or the on-policy shortcut is used. */
#define UNITY_OPT_L2_HINTS_FWD 16 /* 16..19: L2 eviction policy of the forward / recompute / dHidden / dW GEMM: value =
                                     A-operand loads | B-operand loads << 2 | logit-gradient stores << 4, each 0 normal,
                                     1 evict first, 2 evict last (defaults 6, 22, 0, 0: measured +0.3-0.7 % on the first two) */
#define UNITY_OPT_SYNC_PERIOD_GRAD 22 /* 22..24: the recompute / dHidden / dW GEMM's workers meet at every n-th tile (see         */
#define UNITY_OPT_SYNC_PERIOD_DH 23   /* UNITY_OPT_CHUNK_SYNC); 1 = every tile                                                  */
#define UNITY_OPT_SYNC_PERIOD_DW 24
#define UNITY_OPT_HOST_COUNTS 25    /* The kernels of unity_logprob_fwd and unity_ppo_loss_fwd_bwd read the per-model row counts on the
                                     device.  0 (default): the calls never synchronise; the host walks every chunk a model could
                                     have and a launch without rows returns at once.  1: the host reads the K counts back as well
                                     (one stream synchronisation after the routing kernels) and skips the launches that would be
                                     empty (0.1-0.9 % faster on the measured workloads).  Same results either way. */
#define UNITY_OPT_GRAD_ROUNDS 26    /* Schedule of the recompute GEMM.  0: one output tile per unit, workers stride over the tiles
                                     in raster groups and meet at every tile.  n > 0: the forward kernel's schedule: a round =
                                     at most n 128-row tiles x vocabulary splits of the launch's columns, a worker sweeps the
                                     tiles of its split with one row tile and the workers meet once per round.  -1 (default):
                                     rounds of half the SMs where UNITY_OPT_FWD_GROUP's rule allows them (H <= 2368), else 0. */
#define UNITY_OPT_GRAD_BLOCK 27     /* one recompute launch covers value x 18944 rows and vocabulary entries of the gradient
                                     chunk per side; 0 (default): the whole chunk when it runs in rounds or runs of tiles, else 1 */
#define UNITY_OPT_GRAD_RUNS 28      /* The recompute GEMM outside rounds.  0: a unit is one output tile.  n > 0: a unit is a run of column
                                     tiles of one row tile; the kernel cuts the launch's columns into the number of runs that fills
                                     its workers best while about n 128-row tiles are in flight.  -1 (default): n = the tiles whose
                                     hidden rows fit a 45 MB share of L2. */
#define UNITY_OPT_DW_TAIL 29        /* 1 (default): when the vocabulary tiles of a gradient chunk leave a remainder that would fill
                                     less than half of one more wave of CTA pairs, the dW GEMM runs those tiles as a second
                                     launch with narrow column tiles spread over the machine.  0: one launch per chunk. */
#define UNITY_OPT_WAIT_KCYCLES 20  /* bound of every in-kernel wait in thousands of SM clocks (default 4 000 000, about 2 s); when
                                     it runs out the kernel records UNITY_ERR_TIMEOUT, frees its tensor memory and returns */
#define UNITY_OPT_TEST_DROP_SLAB 21 /* TEST HOOK for the timeout path; accepted only while UNITY_OPT_WAIT_KCYCLES <= 1000.
                                     value = 1 + UNITY_PROF_* class: in that class's launches every worker's TMA producer
                                     leaves out one K slab of its first tile, so the waits behind it expire, the launch
                                     returns within milliseconds and unity_check_status reports UNITY_ERR_TIMEOUT (outputs
                                     of that call are undefined).  0 switches it off, and so does a larger wait bound. */
int unity_set_option(unity_ctx* ctx, int option, int value);
int unity_get_profile(unity_ctx* ctx, double* ms, int64_t* launches);

/* ------------------------------------------------------------------------------------------------
 * Stage 1: role-level advantage.
 *
 * Per role invocation s with role v: r_s = lam[v][0]*r_node[s] + lam[v][1]*r_turn[s] +
 * lam[v][2]*r_traj[inv_traj[s]]  - the additive node / turn / trajectory combination of Section
 * "Agent-Specific Reward Interface" (the lambda-weighted equation), rewards being attributed to role
 * invocations (Section "Optimization Objective and System Interface").  Then, per segment
 * (rollout group g, role v) - role identity is kept even when roles share one model (Section
 * "Parameter Sharing in the System") - with n members, mean mu and sigma = sqrt(sum (r-mu)^2 /
 * (n-ddof)):  A_s = (r_s - mu) / (sigma + eps), and A_s = 0 when n-ddof <= 0 or sigma+eps == 0.
 * Finally adv_tok[i] = A_{inv(i)} * tok_mask[i] for every response token of the invocation
 * (paragraph "Batch construction": delayed rewards are aligned with token sequences).
 *
 *   inv_role, inv_group, inv_traj : int32 [n_inv]; an id out of range flags UNITY_ERR_BAD_INDEX and
 *                                   the invocation is left out of the statistics with A = 0
 *   r_node, r_turn : f32 [n_inv] or NULL (= 0);  r_traj : f32 [n_traj] or NULL (= 0)
 *   lam            : (host) f32 [n_roles*3] (node, turn, traj) or NULL (= all 1)
 *   cu_seqlens     : int64 [n_inv+1], non-decreasing, cu_seqlens[0] = 0, cu_seqlens[n_inv] = n_tok
 *   tok_mask       : u8 [n_tok] or NULL (= all 1)
 *   adv_inv        : out f32 [n_inv];  adv_tok : out f32 [n_tok] (NULL allowed when n_tok == 0)
 *   seg_mean, seg_std : out f32 [n_groups*n_roles] or NULL; index g*n_roles+v; 0 for empty segments
 * The members of a segment may sit anywhere in the batch (buffers fill in arrival order): the cost is O(n_inv)
 * whatever the order.  Sums are taken exactly on a per-segment integer grid with integer atomics, so the result
 * does not depend on scheduling (bitwise reproducible; no floating-point atomics), and a segment whose rewards
 * are all equal gets exactly 0.
 * Workspace: unity_advantage_workspace_bytes(n_inv, n_groups, n_roles), about 8 bytes per invocation + 32 bytes per
 * (group, role) segment; n_groups*n_roles <= 2^24.
 */
typedef struct {
    float eps; /* default 1e-6 */
    int ddof;  /* 0 (population) or 1 (sample) */
} unity_adv_params;

size_t unity_advantage_workspace_bytes(int32_t n_inv, int32_t n_groups, int32_t n_roles);
int unity_role_advantage(unity_ctx* ctx, int32_t n_inv, int32_t n_traj, int32_t n_roles, int32_t n_groups,
                         const int32_t* inv_role, const int32_t* inv_group, const int32_t* inv_traj,
                         const float* r_node, const float* r_turn, const float* r_traj, const float* lam,
                         const unity_adv_params* params, int64_t n_tok, const int64_t* cu_seqlens,
                         const uint8_t* tok_mask, float* adv_inv, float* adv_tok, float* seg_mean, float* seg_std);

/* Turn-level reward assembly - the step before stage 1 (paragraph "Reward assembly and commitment"), for the
 * turn-level rules of Section "Workflows and Rewards".  score[j*max_turns + t] is the score after turn t of
 * trajectory j (answer F1 in the iterative search workflow, verifier pass rate in the reflective code workflow);
 * n_scores[j] turns of trajectory j have a score.  Each role v has a rule: with u = inv_turn[s] + rules[v].shift,
 *   UNITY_RULE_ABSOLUTE : r_turn[s] = score[j, u]                 (planner F1(a_0); answer agent F1(a_t))
 *   UNITY_RULE_MARGINAL : r_turn[s] = score[j, u] - score[j, u-1] (loop agents F1(a_t) - F1(a_{t-1}); code workflow
 *                         s_0, s_1 - s_0, s_2 - s_1, with shift = 1 for the reflector, which is paid the next
 *                         round's improvement); the score before the first turn counts as 0
 *   UNITY_RULE_NONE     : r_turn[s] = 0                           (workflows whose roles share only a final score)
 * No score at u, or inv_end[s] != 0 (the agent ended the loop), gives 0.  Shared final scores and node-level format
 * terms need no assembly: they enter stage 1 as r_traj and r_node.
 *   inv_role, inv_traj, inv_turn : int32 [n_inv];  score : f32 [n_traj*max_turns];  n_scores : int32 [n_traj] or
 *   NULL (= max_turns);  inv_end : u8 [n_inv] or NULL;  rules : (host) [n_roles];  r_turn : out f32 [n_inv]
 * An out-of-range role or trajectory id flags UNITY_ERR_BAD_INDEX and yields 0. */
#define UNITY_RULE_NONE 0
#define UNITY_RULE_ABSOLUTE 1
#define UNITY_RULE_MARGINAL 2
typedef struct {
    int mode;  /* UNITY_RULE_* */
    int shift; /* turn offset of the score this role is paid for (0, or 1 for "next round") */
} unity_reward_rule;
int unity_reward_assembly(unity_ctx* ctx, int32_t n_inv, int32_t n_traj, int32_t n_roles, int32_t max_turns,
                          const int32_t* inv_role, const int32_t* inv_traj, const int32_t* inv_turn, const float* score,
                          const int32_t* n_scores, const uint8_t* inv_end, const unity_reward_rule* rules,
                          float* r_turn);

/* Token-level generalized advantage estimation - the advantage formula printed in paragraph "Advantage
 * computation and policy evaluation":  A_t = sum_{l=0}^{T-t} (gamma*lambda)^l delta_{t+l},
 * delta_t = r_t + gamma*V(s_{t+1}) - V(s_t), evaluated per sequence (cu_seqlens) with V = 0 past the last token;
 * returns[t] = A_t + V(s_t) are the regression targets of the value estimates.  Tokens with tok_mask == 0 are not
 * part of their sequence (the next token of t is the next unmasked one) and receive 0 in both outputs.
 *   rewards, values : f32 [n_tok];  tok_mask : u8 [n_tok] or NULL;  gamma, lambda in [0, 1]
 *   advantages, returns : out f32 [n_tok]
 * Uses no workspace; fp32 with a fixed evaluation order (bitwise reproducible). */
int unity_gae(unity_ctx* ctx, int32_t n_inv, int64_t n_tok, const int64_t* cu_seqlens, const float* rewards,
              const float* values, const uint8_t* tok_mask, float gamma, float lambda, float* advantages,
              float* returns);

/* Critic side of the update (paragraph "Model-specific updates and synchronization": each worker group updates its
 * own actor and critic; the quantities are the "value estimates" and "returns" of paragraph "Advantage computation
 * and policy evaluation", returns being unity_gae's second output).  The paper prints no value loss; the one used is
 * PPO's clipped value regression.  Per valid token, with d = v - old_v:
 *   v_clip = v if |d| <= clip_v else old_v + sign(d)*clip_v
 *   l = 0.5 * max((v - R)^2, (v_clip - R)^2)         (equal squares take the unclipped branch)
 *   loss[k] = (1/M_k) sum_{valid tokens of model k} l ,  M_k = norm[k] if given else max(#valid tokens, 1)
 *   dvalues[i] = d loss[model(i)] / d v_i = (v - R)/M_k on the unclipped branch, 0 on the clipped one
 * A token's model is role_model[inv_role[s]] of its invocation s, as in stages 2 and 3.
 *   values, old_values, returns : f32 [n_tok];  tok_mask : u8 [n_tok] or NULL
 *   role_model : (host) int32 [n_roles];  norm : (host) f32 [K] or NULL;  clip_v >= 0 (a huge value disables clipping)
 *   loss : out f32 [K];  clip_frac : out f32 [K] or NULL (share of valid tokens on the clipped branch)
 *   tok_loss : out f32 [n_tok] or NULL;  dvalues : out f32 [n_tok]; masked tokens receive 0 in both
 * An out-of-range role or model id flags UNITY_ERR_BAD_INDEX and the invocation's tokens count as masked.
 * Needs 12 bytes of workspace per invocation plus 5 KiB.  Deterministic (fixed-order sums of floating-point values, integer
 * atomics for the token counts). */
int unity_value_loss_fwd_bwd(unity_ctx* ctx, int32_t n_inv, int32_t n_roles, int32_t K, int64_t n_tok,
                             const int64_t* cu_seqlens, const int32_t* inv_role, const int32_t* role_model,
                             const uint8_t* tok_mask, const float* values, const float* old_values,
                             const float* returns, float clip_v, const float* norm, float* loss, float* clip_frac,
                             float* tok_loss, float* dvalues);

/* Ready-batch construction - the step between a model-local buffer and the update calls (Section "Model-Local
 * Buffers": a buffer becomes a ready-to-update batch by filtering incomplete trajectories, aligning delayed rewards
 * with token sequences, padding, shuffling and matching the data-parallel configuration of the worker group; batches
 * are built per model).  unity_ready_batch_plan decides WHICH invocations enter, in what order and where their tokens
 * go; unity_ready_batch_gather then moves any token-level tensor of the buffer into that order.
 *
 * Plan.  (1) shuffle: position p = 0..n_inv-1 holds invocation perm(p), perm being a seeded bijection of [0, n_inv):
 * four balanced Feistel rounds on the smallest even-width bit domain holding n_inv, applied again while the value is
 * >= n_inv; round function fmix32(right ^ key_i) truncated to the half width, fmix32 = MurmurHash3's 32-bit finaliser,
 * key_i = fmix32(seed32 + 0x9E3779B9*(i+1)), seed32 = low word of seed xor high word.  (2) filter: an invocation is
 * kept when traj_done[inv_traj] != 0 and role_model[inv_role] >= 0 (-1 marks a role that is not trained).  (3) kept
 * invocations are listed model by model, in shuffled order inside a model.  (4) each occupies its length rounded up
 * to a multiple of pad_to.  (5) inside model k, invocation j with P_j padded tokens of the model before it belongs to
 * partition min(n_parts-1, P_j*n_parts / T_k), T_k the model's padded total: contiguous partitions, equal in tokens up
 * to one invocation - one per data-parallel rank or micro-batch.
 *   cu_seqlens : int64 [n_inv+1];  inv_role, inv_traj : int32 [n_inv];  traj_done : u8 [n_traj]
 *   role_model : (host) int32 [n_roles], values in [-1, K)
 *   order          : out int32 [n_inv]: buffer index of the j-th listed invocation; -1 beyond the kept ones
 *   out_cu_seqlens : out int64 [n_inv+1]: padded token offsets in the ready batch; entries beyond the kept ones
 *                    repeat the total
 *   model_offsets  : out int32 [K+1] into order;  part_offsets : out int32 [K*n_parts+1] into order
 *   totals         : out int64 [2]: kept invocations, padded tokens (read it back to size later calls, or size them
 *                    by the bounds n_inv and n_tok + n_inv*(pad_to-1))
 * An out-of-range role or trajectory id drops the invocation and flags UNITY_ERR_BAD_INDEX.  Workspace: about
 * 5 bytes per invocation + 12*K bytes per 256 invocations.  Integer work only: bit-exact and reproducible. */
typedef struct {
    uint64_t seed;
    int32_t n_parts; /* >= 1, <= 65536 */
    int32_t pad_to;  /* >= 1 */
} unity_batch_params;
int unity_ready_batch_plan(unity_ctx* ctx, int32_t n_inv, int32_t n_traj, int32_t n_roles, int32_t K,
                           const int64_t* cu_seqlens, const int32_t* inv_role, const int32_t* inv_traj,
                           const uint8_t* traj_done, const int32_t* role_model, const unity_batch_params* params,
                           int32_t* order, int64_t* out_cu_seqlens, int32_t* model_offsets, int32_t* part_offsets,
                           int64_t* totals);

/* Move a token-level tensor (row_bytes bytes per token: 4 for ids / log-probs / values, 1 for masks, 2*H for hidden
 * rows) from buffer order into the planned order.  The tokens of listed invocation j go to rows out_cu_seqlens[j]..,
 * followed by pad rows up to out_cu_seqlens[j+1] filled with the pad pattern (pad_bytes in {1,2,4,8} dividing
 * row_bytes; pad_value NULL = zeros).
 *   n_inv : size of order;  order, out_cu_seqlens, totals : as written by unity_ready_batch_plan (device)
 *   src_cu_seqlens : int64 [n_inv+1] of the buffer;  src : buffer tensor;  dst : out, at least totals[1] rows
 *   src and dst must be aligned to min(16, largest power of two dividing row_bytes), else UNITY_ERR_ALIGNMENT. */
int unity_ready_batch_gather(unity_ctx* ctx, int32_t n_inv, int64_t n_tok_src, const int32_t* order,
                             const int64_t* src_cu_seqlens, const int64_t* out_cu_seqlens, const int64_t* totals,
                             int64_t row_bytes, const void* src, void* dst, const void* pad_value, int32_t pad_bytes);

/* Delayed rewards (paragraph "Batch construction": trajectory-level or delayed rewards are aligned with the token
 * sequences): tok_reward[t] = r_inv[s] on the last unmasked token of invocation s and 0 on every other token - the
 * reward sequence unity_gae consumes.  An invocation without an unmasked token has no place for its reward.
 *   cu_seqlens : int64 [n_inv+1];  tok_mask : u8 [n_tok] or NULL;  r_inv : f32 [n_inv];  tok_reward : out f32 [n_tok] */
int unity_align_rewards(unity_ctx* ctx, int32_t n_inv, int64_t n_tok, const int64_t* cu_seqlens,
                        const uint8_t* tok_mask, const float* r_inv, float* tok_reward);

/* Stage 1 without any allocation (the paper has no counterpart; this exists for deployment reasons).
 *
 * Who needs it: hosts that may not call cudaMalloc or create a unity_ctx - a trainer whose framework
 * allocator already owns all device memory, a plug-in held to a memory budget by its host process, or a
 * caller that cannot afford the device-wide synchronisation an allocation implies.  The result is the same
 * as unity_role_advantage's (same kernels, same cost O(n_inv)); the scratch (combined reward and segment id per
 * invocation, 32 bytes of accumulators per segment) sits in a fixed device array inside the library instead of a
 * workspace, so no context and no workspace are involved and the call itself performs no cudaMalloc / cudaFree,
 * nor any library routine that allocates.
 *
 *   device, cuda_stream : GPU to run on (made current by the call) and the stream to enqueue on
 *   n_inv               : at most UNITY_NOALLOC_MAX_INV, and n_groups*n_roles at most UNITY_NOALLOC_MAX_SEG,
 *                         otherwise UNITY_ERR_SHAPE (nothing is launched)
 *   bad_index_out       : optional DEVICE int32; receives non-zero (stream-ordered, no sync) when a role,
 *                         group or trajectory id was out of range and its invocation was left out
 *   err, err_len        : optional HOST buffer that receives a one-line reason when the return is not 0
 *   every other argument: exactly as in unity_role_advantage
 * Cost: each GPU that loads the library holds the array (512 B + 8 B * UNITY_NOALLOC_MAX_INV + 32 B *
 * UNITY_NOALLOC_MAX_SEG, about 2.5 MiB) until the process exits.  The first call on a device looks the array's
 * address up (cudaGetSymbolAddress) and may make the CUDA runtime load this library's device code, which is the
 * runtime's own one-time allocation: make that first call outside any stream capture, and count on "no
 * allocation" from the second call on.  The address is kept for the life of the process: do not call
 * cudaDeviceReset while the library is in use.  All calls on a device share the one array and it keeps the
 * previous call's contents - the call clears what must start at zero, but two calls whose kernels can overlap on
 * the GPU (different streams, no ordering between them) race on it: serialise them.
 */
#define UNITY_NOALLOC_MAX_INV 65536
#define UNITY_NOALLOC_MAX_SEG 65536
int unity_role_advantage_noalloc(int device, void* cuda_stream, int32_t n_inv, int32_t n_traj, int32_t n_roles,
                                 int32_t n_groups, const int32_t* inv_role, const int32_t* inv_group,
                                 const int32_t* inv_traj, const float* r_node, const float* r_turn,
                                 const float* r_traj, const float* lam, const unity_adv_params* params,
                                 int64_t n_tok, const int64_t* cu_seqlens, const uint8_t* tok_mask, float* adv_inv,
                                 float* adv_tok, float* seg_mean, float* seg_std, int32_t* bad_index_out, char* err,
                                 size_t err_len);

/* ------------------------------------------------------------------------------------------------
 * Shared description of the response-token rows for stages 2 and 3.  Token i belongs to the
 * invocation s with cu_seqlens[s] <= i < cu_seqlens[s+1]; its role is inv_role[s]; the model that
 * serves it is role_model[role] - the agent-to-model mapping phi of Section "Agent--LLM Mapping"
 * (full sharing, partial sharing, full separation are just different tables).
 */
typedef struct {
    int64_t n_tok;
    int32_t H, V, K, n_inv, n_roles;
    const void* hidden;          /* bf16 [n_tok, H] row-major                                   */
    const void* const* W;        /* (host) K device pointers, each bf16 [V, H] row-major        */
    const int64_t* cu_seqlens;   /* int64 [n_inv+1]                                             */
    const int32_t* inv_role;     /* int32 [n_inv]                                               */
    const int32_t* role_model;   /* (host) int32 [n_roles], values in [0, K)                    */
    const int32_t* target;       /* int32 [n_tok], 0 <= target < V (else BAD_INDEX, row masked) */
    const uint8_t* tok_mask;     /* u8 [n_tok] or NULL (= all 1)                                */
    float inv_temperature;       /* logits are multiplied by this; must be > 0; default 1       */
} unity_rows;

/* Stage 2: the log-probabilities every worker group evaluates for the old, reference and current
 * policy (paragraph "Advantage computation and policy evaluation").  For each valid row, with
 * z = inv_temperature * W_{model(i)} h_i over the whole vocabulary:
 *   lse = log sum_v exp z_v ;  logp[i] = z_target - lse ;  entropy[i] = - sum_v p_v log p_v.
 * The logits exist only in tensor memory; nothing of size n_tok x V is written.
 *   logp : out f32 [n_tok];  entropy, lse : out f32 [n_tok] or NULL.
 */
int unity_logprob_fwd(unity_ctx* ctx, const unity_rows* rows, float* logp, float* entropy, float* lse);

/* Stage 3: the PPO-style policy update of one batch (Section "PPO-Style Training Loop"; paragraph
 * "Model-specific updates and synchronization": each model has its own loss and gradients).
 * Per valid row, with logp and entropy H as in stage 2 and rho = exp(logp - old_logp):
 *   pg  = max(-rho*A, -clip(rho, 1-clip_lo, 1+clip_hi)*A)            (ties take the unclipped branch)
 *   d   = ref_logp - logp ;  kl = -d (mode 1) | d*d/2 (mode 2) | exp(d)-d-1 (mode 3)
 *   l_i = pg + kl_coef*kl - ent_coef*H
 *   loss[k] = (1/M_k) sum_{valid i of model k} l_i ,  M_k = norm[k] if given else max(#valid rows, 1)
 * Backward: dHidden[i,:] = dL/dh_i (bf16, zeros on masked rows) and dW[k] = dL/dW_k (f32), where the
 * logits are recomputed per vocabulary chunk; only a bounded chunk of logit gradients is ever stored.
 *   old_logp, ref_logp, adv_tok : f32 [n_tok]
 *   loss     : out f32 [K]
 *   metrics  : out f32 [(K + n_roles) * UNITY_N_METRICS] or NULL: K per-model records then n_roles
 *              per-role records (role metrics stay separate under parameter sharing)
 *   logp, entropy, tok_loss : out f32 [n_tok] or NULL
 *   dHidden  : out bf16 [n_tok, H];  dW : (host) K device pointers, each f32 [V, H]
 * norm + accumulate_dW make gradient accumulation over micro-batches exact.
 * Deterministic: no floating-point atomics anywhere.
 */
typedef struct {
    float clip_lo, clip_hi; /* 0.2, 0.2 */
    float kl_coef;
    int kl_mode;            /* 1, 2 or 3 (default 3) */
    float ent_coef;
    const float* norm;      /* (host) f32 [K] or NULL */
    int accumulate_dW;      /* 0: overwrite dW, 1: add to it */
    /* On-policy shortcut (all three or none; device f32 [n_tok]): logp, entropy and lse that unity_logprob_fwd
     * returned for THESE weights on THESE rows - e.g. the "old log probabilities" pass of the first PPO epoch, when
     * the current policy still equals the old one.  The forward sweep over the vocabulary is then skipped (2*H*V of
     * the 8*H*V flop per token); the backward still recomputes the logits per chunk.  NULL: full computation. */
    const float* logp_in;
    const float* entropy_in;
    const float* lse_in;
} unity_ppo_params;

int unity_ppo_loss_fwd_bwd(unity_ctx* ctx, const unity_rows* rows, const unity_ppo_params* params,
                           const float* old_logp, const float* ref_logp, const float* adv_tok, float* loss,
                           float* metrics, float* logp, float* entropy, float* tok_loss, void* dHidden,
                           void* const* dW);

#ifdef __cplusplus
}
#endif
#endif /* UNITY_H_ */
