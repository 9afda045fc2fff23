/*
 * entropyinfer.h -- C ABI of the B200 (sm_100a) EntropyInfer prefill path:
 * entropy-guided, head- and segment-adaptive block-sparse causal GQA attention.
 *
 * The path has four stages (paper: "Entropy-Guided Sparse Prefill", Algorithms 1-3,
 * and the complexity appendix, Eqs. t_obs / t_topk / t_spa):
 *   1. pooled representatives of Q and K (Alg. 1), observation attention A_obs
 *      (Alg. 2) and its row entropy e[h,i] per query head h and query segment i;
 *   2. head class (Rigid when max_i e[h,i] < e_t) and per-(head, segment) budgets
 *      from the entropy-fluctuation recurrence (Alg. 3), turned into key-block counts;
 *   3. top-k key blocks per (head, segment) by A_obs (Eq. t_topk), diagonal blocks
 *      always kept, ties to the lower block index;
 *   4. causal softmax attention over the selected key blocks only (Eq. t_spa).
 *
 * Conventions
 *   - q, k, v, out are CALLER-OWNED DEVICE pointers to bf16; the innermost
 *     (head_dim) axis is contiguous; head and token strides are in elements.
 *     Base addresses and strides*2 must be multiples of 16 bytes.
 *   - Every call enqueues work on the given CUDA stream (a cudaStream_t passed as
 *     void*) and returns without synchronising, unless stated otherwise.
 *   - The library owns the plan object and all of its device storage.
 *   - Every function returns EI_OK (0) or a negative ei_status; nothing throws,
 *     aborts or traps.  Device-side waits are bounded: a wait that runs out sets
 *     the plan's device status word (read it with ei_plan_status).
 *   - A plan is one unit of scratch: calls on the same plan must be ordered (one host thread at a time, work on
 *     one stream or streams the caller orders); different plans are independent.  A plan belongs to the device
 *     that was current at ei_plan_create; launching calls made with another device current return
 *     EI_ERR_WRONG_DEVICE.
 *   - One GPU per plan; batches as stacked heads (equal lengths) or ei_prefill_varlen (packed, unequal lengths).
 *     Requires an sm_100 device; there is no CPU fallback.
 */
#ifndef ENTROPYINFER_H_
#define ENTROPYINFER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum ei_status {
  EI_OK = 0,
  EI_ERR_INVALID_ARG = -1,       /* null pointer, bad struct_size, bad enum                     */
  EI_ERR_UNSUPPORTED_SHAPE = -2, /* head_dim not in {64,128,256}, block_len not in {64,128},
                                    (seq_len - q_len) % block_len, segment_len % block_len,
                                    n_q_heads % n_kv_heads, segment_len % 128, misaligned strides,
                                    more causal blocks per row than the scoring kernel can stage */
  EI_ERR_BUDGET_INFEASIBLE = -3, /* total below the forced diagonal count or above all blocks   */
  EI_ERR_ARCH = -4,              /* device is not sm_100                                        */
  EI_ERR_ALLOC = -5,             /* device or host allocation failed                            */
  EI_ERR_CUDA = -6,              /* a CUDA runtime / driver call failed                         */
  EI_ERR_DEVICE_TIMEOUT = -7,    /* a bounded device-side wait ran out                          */
  EI_ERR_PLAN_MISMATCH = -8,     /* imported lists inconsistent with the plan's shape           */
  EI_ERR_NOT_PLANNED = -9,       /* ei_sparse_prefill before ei_plan / ei_plan_set_lists        */
  EI_ERR_SCRATCH_TOO_SMALL = -10, /* ei_entropy_noalloc: the shape needs more than the fixed scratch */
  EI_ERR_WRONG_DEVICE = -11      /* a launching call was made with another device current than at ei_plan_create */
} ei_status;

typedef enum ei_budget_mode {
  /* Paper-faithful: base budget B_h in tokens (Alg. 3; the paper uses 2048), no fixed total.  */
  EI_BUDGET_BASE_TOKENS = 0,
  /* Benchmark configs: the base budget is solved for so that the block counts sum exactly to
     T = floor(budget_fraction * H * sum_i C_i + 0.5), C_i = (segment_len/block_len)*(i+1).     */
  EI_BUDGET_TOTAL_FRACTION = 1
} ei_budget_mode;

/* Problem description and hyper-parameters (Key Notations; Alg. 3 constants).               */
typedef struct ei_params {
  uint32_t struct_size;        /* sizeof(ei_params), for versioning                            */
  int32_t n_q_heads;           /* H                                                            */
  int32_t n_kv_heads;          /* H_kv; query head h reads KV head h / (H / H_kv)              */
  int32_t head_dim;            /* d: 64, 128 or 256 (256: planning in two passes over d, one-tile attention kernel).
                                  Other widths (96, 192) return EI_ERR_UNSUPPORTED_SHAPE, by design: a row of
                                  Q / K is streamed as a power-of-two number of 16-byte lanes (pooling gives each
                                  lane one thread of a power-of-two team and reduces the team by shuffles), the
                                  fp64 observation kernel stages d in 64-wide passes of a fixed count, and the
                                  attention kernels lay the operands out as whole pairs of 64-column swizzled
                                  panels with O in a power-of-two tensor-memory allocation (a 192-wide O next to
                                  S leaves no room for the second tile).  Pad such heads to the next supported
                                  width with zero columns: logits, entropies, selections and outputs are
                                  unchanged (the added output columns are zero) when obs_scale and attn_scale are
                                  given as 1/sqrt(true d).                                                    */
  int32_t seq_len;             /* N; need not be a multiple of segment_len or block_len: there are then
                                  C_S = ceil(N/L_S) segments and C_B = ceil(N/L_B) key blocks, the short
                                  last segment / block is pooled over the rows it has, segment i sees
                                  C_i = min(r(i+1), C_B) blocks (a case the paper does not treat)          */
  int32_t segment_len;         /* L_S: query segment; multiple of block_len and of 128         */
  int32_t block_len;           /* L_B: key block; 64 or 128                                    */
  int32_t budget_mode;         /* ei_budget_mode                                               */
  int64_t q_stride_head, q_stride_tok; /* element strides of q [H, N, d]                       */
  int64_t k_stride_head, k_stride_tok; /* of k [H_kv, N, d]                                    */
  int64_t v_stride_head, v_stride_tok; /* of v [H_kv, N, d]                                    */
  int64_t o_stride_head, o_stride_tok; /* of out [H, N, d]                                     */
  double base_budget_tokens;   /* B_h (BASE mode)                                              */
  double budget_fraction;      /* f in (0,1] (TOTAL mode)                                      */
  double entropy_threshold;    /* e_t, paper 1e-5                                              */
  double alpha;                /* budget coefficient, paper 0.5                                */
  double delta_t;              /* fluctuation threshold, paper 0.4                             */
  double max_mult;             /* budget cap in units of B_h, paper 3; 1 <= max_mult <= 64     */
  double obs_scale;            /* logit scale of Alg. 2; <= 0 selects 1/sqrt(d)                */
  double attn_scale;           /* logit scale of the attention; <= 0 selects 1/sqrt(d)         */
  uint32_t flags;              /* ei_flags                                                     */
  uint32_t q_len;              /* 0: whole prefill, q has seq_len rows.  Otherwise (a later chunk of a chunked
                                  prefill, queries are a suffix of the keys): q and out have q_len rows, which
                                  are the LAST q_len of the seq_len key positions; seq_len - q_len must be a
                                  multiple of block_len.  Segments are counted from the chunk's first row;
                                  segment i sees the blocks below position seq_len - q_len + (i+1) L_S; the
                                  Alg. 3 recurrence starts afresh at the chunk's first segment.  K is pooled
                                  over all seq_len keys on every call.  (The paper treats one-shot prefill
                                  only; this is the same computation restricted to the chunk's rows.)      */
} ei_params;

typedef enum ei_flags {
  EI_FLAG_NONE = 0,
  /* Diagnostic: stage the probabilities P through shared memory for the P.V product instead of
     keeping them in tensor memory.  Same result, slower.                                       */
  EI_FLAG_ATTN_P_VIA_SMEM = 1u << 0,
  /* Use the attention kernel that gives each CTA one 128-row query tile even where the segment
     length would allow the faster two-tile kernel.                                             */
  EI_FLAG_ATTN_SINGLE_TILE = 1u << 1,
  /* Use the two-tile kernel with one softmax thread per query row even where the faster kernel with
     two threads per row applies (head_dim 128, block_len 128).                                  */
  EI_FLAG_ATTN_PAIR_8WARP = 1u << 2,
  /* Group-shared planning (the "Averaged" aggregation of the entropy-pattern figure: attention entropies
     aggregated per GQA group): the G = H / H_kv query heads of a KV head get one entropy curve
     e_g[i] = mean_h e_h[i] and one block ranking by A_g[i,j] = mean_h A_obs,h[i,j]; class, budgets and lists
     exist once per KV head (the "list heads"), and every query head of the group attends over its group's
     list.  In TOTAL mode T = floor(f * H_kv * sum_i C_i + 0.5).  The paper gives no formula for the
     aggregation; mean of entropies and mean of observation attention are this library's reading.      */
  EI_FLAG_GROUP_SHARED = 1u << 3,
  /* ei_plan normally picks between two equivalent schedules of stages 1a/1b by shape: the four stage kernels
     one after another (as the ei_stage_* calls do), or K pooled alone followed by one persistent kernel
     whose pooling warps stream the queries while its other warps run the observation of the row before
     (used when there are at least four rows of work per SM).  These flags force one or the other.     */
  EI_FLAG_PLAN_STAGED = 1u << 4,
  EI_FLAG_PLAN_FUSED = 1u << 5,
  /* Attention by the persistent form of the two-threads-per-row kernel (head_dim 128, block_len 128, segments a
     multiple of 256): one CTA per SM takes (head, segment, tile pair) items off a counter and keeps its
     barriers, tensor memory and K/V ring across items.  Same result bit for bit; within a few per cent of the
     default form either way (faster in short bursts on short block lists, slower in long runs).            */
  EI_FLAG_ATTN_PERSISTENT = 1u << 6,
  /* stage 4: one CTA per tile pair (the default; kept so that callers can say so explicitly)               */
  EI_FLAG_ATTN_PER_CTA = 1u << 7,
  /* The two-threads-per-row kernels leave out the exponentials of a half row (64 keys of one query) whose
     largest logit lies more than 24 binary orders below the row's running maximum, for whole warps of such
     half rows: those probabilities are below 2^-24 of the row's largest term (the resolution of the fp32
     accumulation) and are set to zero.  Heads whose attention sits on a few keys (the Rigid class) spend
     most key blocks there.  This flag switches the shortcut off: every probability is evaluated.          */
  EI_FLAG_ATTN_NO_SKIP = 1u << 8,
  /* On top of that shortcut (default kernel only): where all eight softmax warps of a 128-row tile wrote zeros
     for a key block, that block's P.V product is not issued either.  It would add exactly nothing, so the
     output is bit-identical; EI_ITEM_STATS counts the products left out.  Off by default so that the tensor-core
     work of a launch does not depend on the data.                                                          */
  EI_FLAG_ATTN_SKIP_ZERO_PV = 1u << 9,
  /* The quad-layout kernels (head_dim 128, block_len 128, segments a multiple of 256): sixteen softmax warps,
     each owning sixteen query rows and all 128 key columns of a block through the 16-lane tensor-memory shapes,
     so that the row maximum needs only two shuffles inside a quad of threads and no exchange between warps;
     per-item records (list offset, visible and masked block counts) are worked out once per plan.  The form with
     one CTA per tile pair is what ei_sparse_prefill runs on these shapes when no attention flag is given.  This
     flag selects the other two forms: with EI_FLAG_ATTN_PERSISTENT one CTA per SM with a scheduler warp and a
     ring of item records, with EI_FLAG_ATTN_SINGLE_TILE one 128-row tile per CTA and two CTAs per SM (both
     bit-identical to the default and a few per cent slower in the measurements kept under profiles/).        */
  EI_FLAG_ATTN_QUAD = 1u << 10,
  /* Attention by the split-row kernel (same shapes; the default before the quad-layout kernel): two softmax threads
     per query row in different warps, which agree on the row maximum through shared memory.  Within a few per
     cent of the default; the only kernel that implements EI_FLAG_ATTN_SKIP_ZERO_PV (which implies it).      */
  EI_FLAG_ATTN_SPLIT = 1u << 11,
  /* Attention by the three-buffer kernel (same shapes): one 128-row tile at a time per CTA with three S buffers
     and one O in tensor memory, Q.K^T three key blocks ahead of P.V, two sets of softmax warps on alternate key
     blocks that pass the row reference maxima to each other through shared memory; a CTA runs through several
     consecutive tiles of a segment.                                                                          */
  EI_FLAG_ATTN_TRI = 1u << 12,
  /* The plan holds a SHARD of the heads of a layer (whole KV groups; the other heads live in plans on other
     GPUs): in TOTAL mode its index buffer is sized for all causal blocks of its heads, because the common total
     is apportioned over the multipliers of ALL heads and a shard may be handed more than its own share.  Such a
     plan is driven by ei_plan_observe, ei_stage_multipliers, (all-gather of the tables), ei_stage_apportion,
     ei_stage_select instead of ei_plan.                                                                     */
  EI_FLAG_HEAD_SHARD = 1u << 13
} ei_flags;

/* Fills *p with the paper's constants (e_t 1e-5, alpha 0.5, delta_t 0.4, cap 3, B_h 2048,
   scales 1/sqrt(d)) and contiguous strides for the given shape; budget_mode = TOTAL with the
   given fraction when fraction > 0, BASE otherwise.                                            */
int ei_params_default(ei_params* p, int n_q_heads, int n_kv_heads, int head_dim, int seq_len,
                      int segment_len, int block_len, double fraction);

typedef struct ei_plan_s ei_plan_t; /* opaque */

/* Validates params, allocates the plan's device storage (entropy table, pooled
   representatives, score matrix, budgets, offsets, index lists) for this shape on the current
   device.  Synchronous; the only call besides ei_plan_destroy and ei_prefill_host that
   allocates.                                                                                   */
int ei_plan_create(const ei_params* params, ei_plan_t** out);
void ei_plan_destroy(ei_plan_t* plan);

/* Stages 1-3 (Alg. 1, Alg. 2 + entropy, Alg. 3 + block budgets, top-k selection): fills the
   plan from q [H,N,d] and k [H_kv,N,d].  v is not read (may be NULL).  Asynchronous.          */
int ei_plan(ei_plan_t* plan, const void* q, const void* k, const void* v, void* stream);

/* Stage 4 (the computation counted by Eq. t_spa): out[h,t,:] = sum_u softmax_u(s q_t.k_u) v_u
   over keys u <= t lying in the key blocks selected for (h, segment of t).  Asynchronous.     */
int ei_sparse_prefill(const ei_plan_t* plan, const void* q, const void* k, const void* v,
                      void* out, void* stream);

/* Whole path from HOST buffers (contiguous [H,N,d] / [H_kv,N,d] bf16; pinned memory lets the copies overlap):
   copies q, k, v to plan-owned device staging (allocated on first use, with two copy streams of the plan's
   own), runs ei_plan once q and k have arrived, then ei_sparse_prefill one KV group at a time as its v
   arrives, each group's output going back to out_host while later groups are still uploaded and attended;
   returns after everything has completed (the stream is synchronised).  Results equal ei_plan +
   ei_sparse_prefill on device copies bit for bit.  In BASE mode, where a head's budgets depend on that head
   alone, every KV group is uploaded, planned, attended and sent back on its own (in per-group plans the call
   creates on first use), so uploads, kernels and downloads of different groups overlap; in that mode the
   plan's own items (ei_plan_read) are not filled by this call.                                   */
int ei_prefill_host(ei_plan_t* plan, const void* q_host, const void* k_host, const void* v_host,
                    void* out_host, void* stream);

/* Producer-side pooling (Section 4.1 pools the query and key tensors; Section 4.4 counts that pass in
   t_obs): the step that WRITES q and k can pool them on the way, which removes the planner's own read of
   both tensors.  This call is such a producer: rotary position embedding in the half-rotation form,
       y[t, j] = x[t, j] cos[p, j] - x[t, j + d/2] sin[p, j],   y[t, j + d/2] = x[t, j + d/2] cos[p, j] + x[t, j] sin[p, j],
   p = the position of token t (key row t: p = t; query row t: p = seq_len - q_len + t), j < d/2, computed in fp32
   and rounded to bf16; cos_table / sin_table are DEVICE fp32 arrays [seq_len, d/2], 16-byte aligned.  q_in / q_out
   and k_in / k_out use the plan's q and k strides and may be the same buffers (in place).  In the same pass the
   max / min representatives (Alg. 1) of the rotated rows are written into the plan, after which ei_plan_pooled
   plans without reading q or k.  Only the key blocks from the plan's k_blocks_valid on (ei_plan_set_lengths) are
   rotated and pooled; earlier rows of k are not touched.  flags: EI_ROPE_NO_POOL leaves the representatives alone
   (the plain producer, for comparison).  Asynchronous.                                                        */
enum { EI_ROPE_NO_POOL = 1 };
int ei_rope_pool(ei_plan_t* plan, const void* q_in, const void* k_in, const float* cos_table, const float* sin_table,
                 void* q_out, void* k_out, uint32_t flags, void* stream);

/* Stages 1b-3 (Alg. 2 + entropy, Alg. 3 + block budgets, top-k selection) from the pooled representatives the plan
   already holds (written by ei_rope_pool, ei_stage_pool or ei_plan_write).  Asynchronous.                      */
int ei_plan_pooled(ei_plan_t* plan, void* stream);

/* Packed batch of sequences of unequal lengths (whole prefills): sequence b holds the token positions
   cu_seqlens_host[b] .. cu_seqlens_host[b+1]-1 along the token axis of q, k, v and out (n_seqs + 1 HOST
   integers, non-decreasing; the tensors use the plan's strides, e.g. head stride = total tokens x d for
   [H, total, d], or token stride = H x d for [total, H, d]).  Every sequence is planned and attended on its own
   -- segments, budgets (TOTAL mode: the plan's fraction of that sequence's causal blocks) and lists never
   cross a sequence boundary -- with the plan re-targeted to its length (ei_plan_set_lengths), so the plan must
   have been created for at least the longest sequence and with q_len = 0.  Results equal one ei_plan +
   ei_sparse_prefill per sequence bit for bit; empty sequences are skipped.  Fails before launching anything
   when a sequence does not fit (EI_ERR_PLAN_MISMATCH), when in TOTAL mode the fraction of a short sequence's
   blocks is below its forced diagonal blocks (EI_ERR_BUDGET_INFEASIBLE; BASE mode has no such limit) or when
   cu_seqlens is not monotone (EI_ERR_INVALID_ARG).
   Launches: sequences whose tables fit the plan's side by side (cells, scores, K representatives, list
   entries: a plan created for the batch's total length, each sequence rounded up to whole segments, holds them
   all; at most 256 at a time) run in ONE set of five launches -- pooling, observation, budget (one CTA per
   sequence), selection, attention -- in which every CTA looks up its sequence in a small table copied to the
   device with the call (group-shared lists: a sixth launch for the aggregation); this applies to every shape
   with the attention kernel the library picks by default.  A sequence that fits only on its own (a plan made
   for the longest sequence), and every sequence of a plan whose flags name another attention kernel, takes the
   plan re-targeted to it and the ordinary two calls (four to five launches per sequence).  The results are the
   same either way.
   Asynchronous; afterwards the plan is targeted at the last non-empty sequence.  It holds that sequence's
   tables when the sequence ran on its own; after a set of packed launches the tables hold the batch, one
   sequence after another, and ei_sparse_prefill returns EI_ERR_NOT_PLANNED until the next ei_plan.          */
int ei_prefill_varlen(ei_plan_t* plan, const void* q, const void* k, const void* v, void* out,
                      const int32_t* cu_seqlens_host, int n_seqs, void* stream);

/* Single stages on the plan's own buffers, for stage-isolated checks (inject inputs with
   ei_plan_write first).  Asynchronous.                                                         */
int ei_stage_pool(ei_plan_t* plan, const void* q, const void* k, void* stream);   /* Alg. 1     */
int ei_stage_observe(ei_plan_t* plan, void* stream);   /* Alg. 2 + entropy, from the pooled reps */
int ei_stage_budget(ei_plan_t* plan, void* stream);    /* Alg. 3 + block counts, from entropy    */
/* Stages 1a + 1b of ei_plan alone (pooling and observation in the plan's schedule): ENTROPY and SCORES.  */
int ei_plan_observe(ei_plan_t* plan, const void* q, const void* k, void* stream);
/* Alg. 3 in its two halves, for a layer whose heads are sharded over several GPUs (one plan per shard, each
   holding whole KV groups; everything of the method is per head except TOTAL mode's common total, which
   couples the heads through the base budget b*):
     ei_stage_multipliers   class and multiplier recurrence of the plan's heads from ENTROPY: CLASS and
                            MULTIPLIERS (M = floor(m*4096 + 0.5), int32 [H, C_S]); when multipliers_out_dev is
                            not NULL the table is also copied there (device, H*C_S int32) -- the send buffer of
                            the all-gather;
     ei_stage_apportion     block counts of the plan's heads as rows [first_head, first_head + H) of the
                            apportionment of total_all blocks over the n_heads_all heads of
                            multipliers_all_dev (device, int32 [n_heads_all, C_S], the gathered tables in head
                            order): the same b*, the same leftover cells as one plan over all heads would find,
                            so the shards' BUDGET rows are the rows of that plan bit for bit.  BASE mode looks
                            at the plan's own rows only.  Writes BUDGET, OFFSETS and STATS (total and extremes
                            of the plan's own heads; b* and leftover of the whole layer).
   Between the two the caller gathers the tables (e.g. ncclAllGather on the same stream); no other exchange is
   needed.  ei_stage_apportion fails with EI_ERR_BUDGET_INFEASIBLE when total_all is below the forced diagonal
   blocks or above all causal blocks of n_heads_all heads, with EI_ERR_PLAN_MISMATCH when the plan's index
   buffer could not hold what it may be handed (create it with EI_FLAG_HEAD_SHARD).  Asynchronous.
   (Related Work: every quantity of the method is per head h; Alg. 3.)                                       */
int ei_stage_multipliers(ei_plan_t* plan, int32_t* multipliers_out_dev, void* stream);
int ei_stage_apportion(ei_plan_t* plan, const int32_t* multipliers_all_dev, int n_heads_all, int first_head,
                       int64_t total_all, void* stream);
int ei_stage_select(ei_plan_t* plan, void* stream);    /* top-k lists, from scores + counts      */

typedef enum ei_item {
  EI_ITEM_ENTROPY = 0, /* float   [H, C_S]                                                      */
  EI_ITEM_CLASS = 1,   /* uint8   [H]           1 = Rigid                                       */
  EI_ITEM_BUDGET = 2,  /* int32   [H, C_S]      key blocks per (head, segment)                  */
  EI_ITEM_OFFSETS = 3, /* int32   [H*C_S + 1]   CSR offsets into INDICES                        */
  EI_ITEM_INDICES = 4, /* int32   [capacity]    block indices, ascending per cell               */
  EI_ITEM_SCORES = 5,  /* float   [H, sum_i C_i] ln A_obs; row i of head h at r*i*(i+1)/2       */
  EI_ITEM_QMAX = 6,    /* bf16    [H, C_S, d]                                                   */
  EI_ITEM_QMIN = 7,
  EI_ITEM_KMAX = 8,    /* bf16    [H_kv, C_B, d]                                                */
  EI_ITEM_KMIN = 9,
  EI_ITEM_STATS = 10,  /* int64   [8]: total blocks, rigid heads, b* (1/4096 block), leftover R,
                                        min k, max k, P.V products (128-row tile x key block) that the
                                        ei_sparse_prefill calls since the last ei_plan left out because P
                                        was all zero (EI_FLAG_ATTN_SKIP_ZERO_PV), reserved      */
  /* With EI_FLAG_GROUP_SHARED the items CLASS, BUDGET, OFFSETS and INDICES above are per list head
     (H_kv of them instead of H); ENTROPY and SCORES stay per query head, and the aggregated tables that
     stages 2 and 3 read are:                                                                    */
  EI_ITEM_GROUP_ENTROPY = 11, /* float [H_kv, C_S]                                              */
  EI_ITEM_GROUP_SCORES = 12,  /* float [H_kv, sum_i C_i] ln A_g                                 */
  EI_ITEM_MULTIPLIERS = 13    /* int32 [H, C_S] (list heads): M = floor(m*4096 + 0.5) of Alg. 3     */
} ei_item;

/* Borrowed device pointer and size in bytes of one plan item; valid until ei_plan_destroy.    */
int ei_plan_get(const ei_plan_t* plan, int item, const void** dev_ptr, size_t* bytes);
/* Copies one item to / from a host buffer of exactly `bytes` (<= the item's size) and
   synchronises the stream.                                                                     */
int ei_plan_read(const ei_plan_t* plan, int item, void* host_dst, size_t bytes, void* stream);
int ei_plan_write(ei_plan_t* plan, int item, const void* host_src, size_t bytes, void* stream);

/* Loads block counts k [H*C_S] and ascending index lists (concatenated in cell order) from the
   host, e.g. made by another implementation.  Validates ranges and order on the host;
   synchronous.                                                                                 */
int ei_plan_set_lists(ei_plan_t* plan, const int32_t* k_host, const int32_t* idx_host,
                      size_t n_idx, void* stream);

/* Re-targets an existing plan, without allocating, to a shorter problem with the same heads, sizes and strides:
   seq_len key positions of which the last q_len are the queries (q_len = 0: all of them; seq_len - q_len a
   multiple of block_len), as a serving loop does that prefills a prompt chunk by chunk into buffers laid out
   for the full length.  k_blocks_valid says how many leading key blocks already have their pooled
   representatives in the plan from earlier ei_plan calls on the same K prefix (pass the number of COMPLETE
   blocks of the previous call's seq_len, or 0): the next ei_plan pools only the blocks from there on.  Fails
   with EI_ERR_PLAN_MISMATCH, leaving the plan unchanged, when the new shape needs more storage than the plan
   was created with.  Host-only; kernels already enqueued keep the shape they were launched with.  Both
   schedules (and ei_stage_pool) skip the pooling of the first k_blocks_valid blocks.                      */
int ei_plan_set_lengths(ei_plan_t* plan, int seq_len, int q_len, int k_blocks_valid);

/* Synchronises the stream and returns the device status word (EI_OK or EI_ERR_DEVICE_TIMEOUT),
   then clears it.                                                                              */
int ei_plan_status(ei_plan_t* plan, void* stream);

/* Testing aid for the error contract above (EI_ERR_DEVICE_TIMEOUT): every device-side wait of the library is
   bounded (2^30 clocks, about half a second) and a wait that runs out sets the plan's status word, after which
   every later wait returns at once, the kernels run to their common end, wait for their own copies in flight,
   free their tensor memory and return.  This call makes that path reachable without a faulty GPU:
   wait_limit_log2 > 0 shortens the bound of the plan's kernels to 2^wait_limit_log2 clocks (0: the default),
   and skip_ring_item >= 0 makes the producer warp of the default stage-4 kernel and of the split-row kernel
   (head_dim 128, block_len 128, segments a multiple of 256) leave out that K/V load of every tile pair (item 2j is K of the j-th listed
   block, 2j + 1 its V; -1: none), so that the consumer's wait for it runs out.  ei_plan_status then reports
   the timeout and clears it; after ei_plan_debug_waits(plan, 0, -1, stream) the plan works as before.
   Host-synchronous on `stream`.  No counterpart in the paper.                                             */
int ei_plan_debug_waits(ei_plan_t* plan, int wait_limit_log2, int skip_ring_item, void* stream);

/* Configured total T (TOTAL mode) or the list capacity (BASE mode).                          */
int64_t ei_plan_total_blocks(const ei_plan_t* plan);
/* Number of kernels this library has launched for the plan so far.                           */
int64_t ei_plan_launches(const ei_plan_t* plan);

/* ---- Follow-on to the prefill path: latent KV-cache compression (appendix "Latent KV Cache Compression
   Algorithm", Algorithm 4; Section 4.3).  After N_D tokens have been generated, the cache of each KV head is
   cut to the B_d positions that the queries of an observation window score highest:
       S = Q_W K^T (raw logits),  w_j = sum_i S[i,j],  keep top-B_d of w,  gather K and V.
   One index set per KV head, scored with all query heads of its group; ties keep the lower position; the
   kept positions come out in increasing order.                                                          */
typedef struct ei_compress_params {
  uint32_t struct_size;                 /* sizeof(ei_compress_params)                                    */
  int32_t n_q_heads, n_kv_heads;        /* H, H_kv                                                       */
  int32_t head_dim;                     /* d: 64, 128 or 256                                             */
  int32_t kv_len;                       /* L: cached positions (prompt + generated so far)               */
  int32_t window;                       /* N_W: rows of q_window per head                                */
  int32_t budget;                       /* B_d: positions kept per KV head (paper: 1024)                 */
  int32_t reserved;
  int64_t q_stride_head, q_stride_tok;  /* q_window [H, N_W, d]: the queries at the window positions     */
  int64_t k_stride_head, k_stride_tok;  /* k [H_kv, L, d]                                                */
  int64_t v_stride_head, v_stride_tok;  /* v [H_kv, L, d]                                                */
} ei_compress_params;

/* Bytes of device workspace ei_latent_compress needs (the score vector w [H_kv, L] float, the summed
   window queries and a per-head histogram); 0 for invalid parameters.                                   */
size_t ei_latent_compress_workspace_bytes(const ei_compress_params* params);

/* All pointers are caller-owned device memory (bf16 tensors, 16-byte aligned; strides in elements, d
   contiguous).  Writes idx_out [H_kv, min(B_d, L)] int32 (ascending), k_out / v_out [H_kv, min(B_d, L), d]
   bf16, and leaves w in the first H_kv*L floats of workspace.  Allocates nothing.  Asynchronous.        */
int ei_latent_compress(const ei_compress_params* params, const void* q_window, const void* k, const void* v,
                       void* workspace, int32_t* idx_out, void* k_out, void* v_out, void* stream);

/* No counterpart in the paper: an allocation-free way to get the entropy table e[h,i] of stage 1
   (pooling + observation attention, same kernels as ei_plan's first two stages).
   For callers that must not allocate device memory: hosts whose own allocator owns all of HBM
   (a library-side cudaMalloc would fail or fragment it) and loops that cannot afford the
   device-wide synchronisation an allocation implies.  The caller passes q [H,N,d], k [H_kv,N,d]
   (device, bf16, strides from params) and entropy_out (device, float [H, C_S]); the scratch
   (pooled representatives and score rows) is a fixed device array of
   EI_NOALLOC_SCRATCH_BYTES (32 MiB) that every context loading this library holds until exit.
   Shapes needing more return EI_ERR_SCRATCH_TOO_SMALL (the 128k Llama-3-8B and Llama-3.1-70B
   layers fit).  No cudaMalloc, cudaFree or other allocating routine is called.
   The first call on a device looks up the array's device address (cudaGetSymbolAddress) and the
   device's architecture (EI_ERR_ARCH unless sm_100, as ei_plan_create reports it); make that first
   call outside any stream capture.  All calls share the one array and it keeps the
   previous call's contents (none of which is read before being rewritten): two calls whose
   kernels overlap on the GPU (different streams, or threads) race.  Asynchronous on `stream`.  */
int ei_entropy_noalloc(const ei_params* params, const void* q, const void* k, float* entropy_out,
                       void* stream);
#define EI_NOALLOC_SCRATCH_BYTES (32u << 20)

const char* ei_status_string(int status);
int ei_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ENTROPYINFER_H_ */
