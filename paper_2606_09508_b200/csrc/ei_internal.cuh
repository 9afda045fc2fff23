// Internal declarations shared by the CUDA translation units of libentropyinfer.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "entropyinfer.h"

namespace ei {

// Shape-derived constants (Key Notations): r = L_S/L_B key blocks per segment.  The queries are the last
// Nq of the N key positions (Nq = N for a whole prefill; a later chunk of a chunked prefill has P = N - Nq
// keys before it, P a multiple of L_B, c0 = P / L_B).  C_S = ceil(Nq/L_S) segments, C_B = ceil(N/L_B) key
// blocks, C_i = min(c0 + r(i+1), C_B) causal blocks of segment i (only a short last segment is clipped), of
// which [c0 + r*i, C_i) are its diagonal blocks; SC = sum_i C_i per head, cells = H*C_S.
struct Shape {
  int H, Hkv, G, d, N, L_S, L_B, r, C_S, C_B;
  int64_t SC, cells;
  int64_t qs_h, qs_t, ks_h, ks_t, vs_h, vs_t, os_h, os_t;
  int Nq, P, c0;  // query rows, key positions before the first query, key blocks before the first query
  int KB_cap;     // key blocks per KV head in the K-representative arrays (their head stride; >= C_B)
  int list_div;  // query head h reads the block list of list head h / list_div (G when lists are per KV group, else 1)
};

// start of segment i's row in the compact score layout: sum_{i' < i} (c0 + r(i'+1))
__host__ __device__ inline int64_t row_offset(const Shape& s, int64_t i) {
  return (int64_t)s.c0 * i + (int64_t)s.r * i * (i + 1) / 2;
}
__host__ __device__ inline int causal_blocks(const Shape& s, int i) {
  const int c = s.c0 + s.r * (i + 1);
  return c < s.C_B ? c : s.C_B;
}

// One sequence of a packed batch that runs in ONE set of launches (ei_prefill_varlen): its shape and where its
// share of every plan table starts.  A planning / attention kernel that is handed such a table looks its CTA's
// sequence up (w_* = CTAs of the earlier sequences in that kernel's grid) and then works on the sequence as if it
// were alone: the tables of the sequences lie one after another, each laid out exactly as a plan of that
// sequence would lay them out.
struct PackedSeq {
  Shape s;           // the sequence's query-head shape
  Shape ls;          // its list-head shape (H := H_kv under group-shared lists, else the same)
  long long tok0;   // first token of the sequence in q, k, v, out
  long long cell0;  // first (query head, segment) cell: entropy, query representatives
  long long lcell0; // first (list head, segment) cell: group entropy, multipliers, counts, stage-4 records
  long long off0;   // first entry of its offsets (list cells + 1 entries per sequence)
  long long sc0;    // first score (per query head)
  long long lsc0;   // first group score (per list head; = sc0 without group-shared lists)
  long long kb0;    // first key block in the K-representative arrays (KV-head stride there: the sequence's own C_B)
  long long idx0;   // first list entry
  long long T;      // TOTAL mode: the sequence's total
  int head0;        // first class entry
  int index;        // position among the sequences of this set of launches (its Stats slot)
  int w_pool, w_obs, w_sel, w_att;
};
constexpr int MAX_PACKED = 256;  // sequences per set of launches
#ifdef __CUDACC__
__device__ __forceinline__ int packed_find(const PackedSeq* pk, int npk, int bid, int PackedSeq::*w) {
  int lo = 0, hi = npk;  // the last sequence whose first CTA is <= bid
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (pk[mid].*w <= bid) lo = mid;
    else hi = mid;
  }
  return lo;
}
#endif

struct Stats {  // EI_ITEM_STATS
  long long total, rigid_heads, b_star, leftover, min_k, max_k, pv_skipped, reserved1;  // pv_skipped: counted by stage 4
};

// parameter validation shared by the entry points (EI_OK or a negative ei_status)
int shape_from_params(const ei_params* p, Shape* s);

// ---- launch wrappers (each returns a cudaError_t from the launch) -----------------------------
// The *_packed forms run one launch over all npk sequences of pk (device array; pk_host the same on the host,
// for the grid sizes); the table pointers are the plan's, the per-sequence offsets come from pk.
cudaError_t launch_pool_packed(const PackedSeq* pk, const PackedSeq* pk_host, int npk, const __nv_bfloat16* q,
                               const __nv_bfloat16* k, __nv_bfloat16* qmax, __nv_bfloat16* qmin, __nv_bfloat16* kmax,
                               __nv_bfloat16* kmin, cudaStream_t st);
cudaError_t launch_observe_packed(const PackedSeq* pk, const PackedSeq* pk_host, int npk, const __nv_bfloat16* qmax,
                                  const __nv_bfloat16* qmin, const __nv_bfloat16* kmax, const __nv_bfloat16* kmin,
                                  double scale, float* scores, float* entropy, cudaStream_t st);
struct BudgetArgs;
void packed_fill_work(PackedSeq* pk_host, int npk);  // fills w_pool, w_obs, w_sel, w_att
cudaError_t launch_budget_packed(const PackedSeq* pk, int npk, const BudgetArgs& a, const float* entropy,
                                 unsigned char* rigid, int* Mfx, int* kblocks, int* offsets, Stats* stats, cudaStream_t st);
// group-shared lists: the aggregation of every sequence's tables, one launch
cudaError_t launch_group_aggregate_packed(const PackedSeq* pk, const PackedSeq* pk_host, int npk, const float* scores,
                                          const float* entropy, float* g_scores, float* g_entropy, cudaStream_t st);
cudaError_t launch_select_packed(const PackedSeq* pk, const PackedSeq* pk_host, int npk, const float* scores,
                                 const int* kblocks, const int* offsets, int* indices, int* items, cudaStream_t st);
cudaError_t launch_pool(const Shape& s, const __nv_bfloat16* q, const __nv_bfloat16* k,
                        __nv_bfloat16* qmax, __nv_bfloat16* qmin, __nv_bfloat16* kmax,
                        __nv_bfloat16* kmin, int first_block, cudaStream_t st);

// rotary embedding of q and k with the pooling folded in (ei_producer.cu); key blocks from first_block on
cudaError_t launch_rope_pool(const Shape& s, const __nv_bfloat16* q_in, const __nv_bfloat16* k_in, const float* cos_t,
                             const float* sin_t, __nv_bfloat16* q_out, __nv_bfloat16* k_out, __nv_bfloat16* qmax,
                             __nv_bfloat16* qmin, __nv_bfloat16* kmax, __nv_bfloat16* kmin, int first_block, bool pool,
                             cudaStream_t st);

// returns cudaErrorInvalidValue when a row does not fit the kernel's shared-memory staging
cudaError_t launch_observe(const Shape& s, const __nv_bfloat16* qmax, const __nv_bfloat16* qmin,
                           const __nv_bfloat16* kmax, const __nv_bfloat16* kmin, double scale,
                           float* scores, float* entropy, cudaStream_t st);
bool observe_shape_supported(const Shape& s);
int observe_ctas_per_row(const Shape& s);  // CTAs per (KV head, segment) row of the observation kernel's grid

// K blocks only (the query cells are then pooled by the fused kernel below)
cudaError_t launch_pool_k(const Shape& s, const __nv_bfloat16* k, __nv_bfloat16* kmax, __nv_bfloat16* kmin,
                          int first_block, cudaStream_t st);  // blocks [first_block, C_B) of every KV head
// stages 1a (queries) + 1b in one persistent kernel: pooling warps run ahead of observation warps
cudaError_t launch_pool_observe(const Shape& s, const __nv_bfloat16* q, const __nv_bfloat16* kmax,
                                const __nv_bfloat16* kmin, __nv_bfloat16* qmax, __nv_bfloat16* qmin, double scale,
                                float* scores, float* entropy, int* status, cudaStream_t st);
bool pool_observe_shape_supported(const Shape& s);

// group-shared planning: e_g = mean over the group's heads of e, lnA_g = ln(mean of exp(lnA))
cudaError_t launch_group_aggregate(const Shape& s, const float* scores, const float* entropy, float* g_scores,
                                   float* g_entropy, cudaStream_t st);

struct BudgetArgs {
  int mode;            // ei_budget_mode
  long long T;         // TOTAL mode target
  long long b_fx_base; // BASE mode base budget, 1/4096 block
  double e_t, alpha, delta_t, max_mult;
  int phase;           // EI_BUDGET_PHASE_*
  int H_all;           // heads the apportionment runs over (the plan's own unless the layer is sharded)
  int first_head;      // where this plan's heads sit among them
};
enum { EI_BUDGET_PHASE_ALL = 0, EI_BUDGET_PHASE_MULTIPLIERS = 1, EI_BUDGET_PHASE_APPORTION = 2 };
// Mall: the multiplier table [H_all, C_S] of EI_BUDGET_PHASE_APPORTION (device; otherwise unused)
cudaError_t launch_budget(const Shape& s, const BudgetArgs& a, const float* entropy,
                          unsigned char* rigid, int* Mfx, const int* Mall, int* kblocks, int* offsets, Stats* stats,
                          cudaStream_t st);

// items (may be null): the stage-4 records of every (cell, tile pair), written by the warp that made the cell's list
cudaError_t launch_select(const Shape& s, const float* scores, const int* kblocks,
                          const int* offsets, int* indices, int* items, cudaStream_t st);

struct AttnArgs {
  const __nv_bfloat16 *q, *k, *v;
  __nv_bfloat16* out;
  const int* offsets;
  const int* indices;
  int* status;
  float scale;
  bool p_via_smem;   // diagnostic: P through shared memory (single-tile kernel)
  bool single_tile;  // force the one-tile-per-CTA kernel
  bool pair_8warp;   // force the two-tile kernel with one softmax thread per row
  bool persistent;   // the persistent form of the split-row kernel (items off a counter)
  bool quad_kernel;  // the quad-layout kernel (ei_attention_quad.cu)
  bool tri_kernel;   // the three-buffer kernel (ei_attention_tri.cu); needs items like the quad-layout kernels
  int tri_tiles;     // tiles per CTA of the three-buffer kernel (0: its default)
  int* sched;        // two ints, zero between launches: next item, CTAs finished
  float skip_log2;   // split-row kernels: half rows more than this many binary orders below the row maximum get P = 0
                     // without being exponentiated (infinity: never)
  long long* pv_skipped;  // device counter: (tile, block) P.V products left out because P was all zero (may be null)
  const int* items;       // per (list cell, tile pair) records of launch_attention_items (quad-layout kernels), shifted like offsets
};
// returns EI_OK or a negative ei_status (tensor-map encoding can fail)
int launch_attention(const Shape& s, const AttnArgs& a, cudaStream_t st);
int launch_attention_quad(const Shape& s, const AttnArgs& a, cudaStream_t st);  // d = 128, L_B = 128, L_S % 256 = 0
int launch_attention_tri(const Shape& s, const AttnArgs& a, cudaStream_t st);   // same shapes
// the per-CTA quad-layout kernel over all sequences of a packed batch (a.q .. a.out: the packed tensors, a.items /
// a.indices: the plan's arrays; offsets and shapes per sequence from pk)
int launch_attention_quad_packed(const PackedSeq* pk, const PackedSeq* pk_host, int npk, long long n_tokens,
                                 const AttnArgs& a, cudaStream_t st);
// any shape: picks the kernel launch_attention would pick without flags and launches it once over all sequences
int launch_attention_packed(const PackedSeq* pk, const PackedSeq* pk_host, int npk, long long n_tokens, const AttnArgs& a,
                            cudaStream_t st);
// one record of 8 ints per (list cell, tile pair) from the plan's lists (ls: the list-head shape); a no-op for
// shapes the tile-pair kernels do not take
cudaError_t launch_attention_items(const Shape& ls, const int* offsets, const int* indices, int* items, cudaStream_t st);

#ifdef __CUDACC__
// Stage-4 record of one (list cell, tile pair): what a CTA has to know about its pair of 128-row query tiles before it
// can start -- where the cell's ascending block list is, how many of its blocks each of the two tiles sees at all
// (n0, n1), from which entry on they need the causal mask (jm0, jm1) and the first block.  Called by a whole warp
// (`list` holds the cell's nlist entries; they may have been written by this warp just before, hence the L2
// loads); lanes 0-7 store the record {off, n0, n1, jm0, jm1, blk0, 0, 0}.
__device__ __forceinline__ void attention_item_record(const Shape& s, int seg, int pr, int off, int nlist,
                                                      const int* list, int* rec, int lane) {
  constexpr int TILE = 128;
  const int BN = s.L_B;
  const long long q0 = (long long)seg * s.L_S + (long long)pr * 2 * TILE;
  int n0 = 0, n1 = 0, jm0 = 0, jm1 = 0, blk0 = 0;
  if (q0 < s.Nq) {  // a pair beyond the sequence (short last segment) keeps n0 = n1 = 0
    // The list is ascending, so the blocks a tile does not see at all, and the blocks that need the causal mask,
    // are suffixes of it: every lane looks at one entry from the tail, ballots count the suffixes.
    int cut1 = 0, cut0 = 0, msk1 = 0, msk0 = 0;
    for (int b0 = 0; b0 < nlist; b0 += 32) {
      const int e = nlist - 1 - b0 - lane;
      const bool in = e >= 0;
      const long long blk = in ? (long long)__ldcg(list + e) : -1;
      const unsigned c1 = __ballot_sync(0xffffffffu, in && blk * BN > q0 + s.P + 2 * TILE - 1);
      const unsigned c0 = __ballot_sync(0xffffffffu, in && blk * BN > q0 + s.P + TILE - 1);
      const unsigned m1 = __ballot_sync(0xffffffffu, in && (blk + 1) * BN - 1 > q0 + TILE + s.P);
      const unsigned m0 = __ballot_sync(0xffffffffu, in && (blk + 1) * BN - 1 > q0 + s.P);
      cut1 += __popc(c1);
      cut0 += __popc(c0);
      msk1 += __popc(m1);
      msk0 += __popc(m0);
      if (m0 != 0xffffffffu) break;  // the widest suffix ended inside this window
    }
    n1 = nlist - cut1;
    n0 = nlist - cut0;
    jm1 = nlist - msk1 < n1 ? nlist - msk1 : n1;
    jm0 = nlist - msk0 < n0 ? nlist - msk0 : n0;
    blk0 = nlist > 0 ? __ldcg(list) : 0;
  }
  if (lane < 8) rec[lane] = lane == 0 ? off : lane == 1 ? n0 : lane == 2 ? n1 : lane == 3 ? jm0 : lane == 4 ? jm1 : lane == 5 ? blk0 : 0;
}
#endif

// bf16 tensor [heads, N, d] (d contiguous) as a 3-D tensor map, box = 64 x box_rows x 1, 128-byte swizzle
bool make_tensor_map(CUtensorMap* tm, const void* ptr, int d, int N, int heads, int64_t tok_stride,
                     int64_t head_stride, int box_rows);

}  // namespace ei
