// C ABI of libentropyinfer: plan object, validation, stage dispatch.  See include/entropyinfer.h.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "ei_internal.cuh"

using ei::Shape;

struct ei_plan_s {
  ei_params params;
  Shape shape;   // per query head: stages 1a/1b and the attention
  Shape lshape;  // per list head: stages 2 and 3 (the same unless the plan is group-shared: then H = H_kv, G = 1)
  // sizes the device storage was allocated for (ei_plan_set_lengths may re-target the plan to anything that fits)
  long long cap_cells, cap_lcells, cap_scores, cap_lscores;
  int k_first;   // first key block ei_plan pools (blocks before it are kept from earlier calls)
  bool group;    // EI_FLAG_GROUP_SHARED
  float *g_entropy, *g_scores;  // aggregated tables (group-shared plans only)
  long long T;          // configured total (TOTAL mode)
  long long b_fx_base;  // BASE mode base budget, 1/4096 block
  long long capacity;   // length of the index buffer
  long long need_idx;   // list entries the current shape and budget can need (<= capacity)
  double obs_scale, attn_scale;
  // device storage
  float* entropy;
  unsigned char* rigid;
  int* Mfx;
  int* kblocks;
  int* offsets;
  int* indices;
  float* scores;
  __nv_bfloat16 *qmax, *qmin, *kmax, *kmin;
  ei::Stats* stats;
  int* status;
  int* sched;  // item counter of the persistent attention kernel
  ei::PackedSeq* pk;  // per-sequence table of a packed batch that runs in one set of launches (MAX_PACKED entries)
  int* items;  // per (list cell, tile pair) records for stage 4, rebuilt when the lists change
  bool items_valid;
  int device;  // the device the plan's storage lives on
  // host-path staging
  __nv_bfloat16 *sq, *sk, *sv, *so;
  size_t stage_nq, stage_nk;  // elements the staging buffers hold
  cudaStream_t up, down;  // the host path's copy streams
  ei_plan_s** sub;        // BASE mode: one plan per KV group, so that whole groups can be pipelined
  cudaEvent_t* ev;        // and its events: start, K and Q uploaded, all downloaded, V of head g, output of group g
  int n_ev;
  bool planned;
  long long launches;
};

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// A plan's buffers belong to the device that was current when it was created; launching on another one would
// hand a kernel pointers it cannot reach.  Every launching entry point checks first.
bool on_plan_device(const ei_plan_t* pl) {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess && dev == pl->device;
}

int validate(const ei_params* p, Shape* s) {
  if (!p || p->struct_size != sizeof(ei_params)) return EI_ERR_INVALID_ARG;
  if (p->budget_mode != EI_BUDGET_BASE_TOKENS && p->budget_mode != EI_BUDGET_TOTAL_FRACTION)
    return EI_ERR_INVALID_ARG;
  if (p->n_q_heads <= 0 || p->n_kv_heads <= 0 || p->seq_len <= 0 || p->segment_len <= 0 || p->block_len <= 0)
    return EI_ERR_INVALID_ARG;
  if (!(p->entropy_threshold >= 0) || !(p->max_mult >= 1.0) || !(p->max_mult <= 64.0) || !isfinite(p->alpha) ||
      !isfinite(p->delta_t))
    return EI_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128 && p->head_dim != 256) return EI_ERR_UNSUPPORTED_SHAPE;
  if (p->block_len != 64 && p->block_len != 128) return EI_ERR_UNSUPPORTED_SHAPE;
  if (p->n_q_heads % p->n_kv_heads) return EI_ERR_UNSUPPORTED_SHAPE;
  if (p->segment_len % p->block_len || p->segment_len % 128) return EI_ERR_UNSUPPORTED_SHAPE;
  const int64_t strides[8] = {p->q_stride_head, p->q_stride_tok, p->k_stride_head, p->k_stride_tok,
                              p->v_stride_head, p->v_stride_tok, p->o_stride_head, p->o_stride_tok};
  for (int64_t st : strides)
    if (st < p->head_dim || st % 8) return EI_ERR_UNSUPPORTED_SHAPE;
  s->H = p->n_q_heads;
  s->Hkv = p->n_kv_heads;
  s->G = s->H / s->Hkv;
  s->d = p->head_dim;
  s->N = p->seq_len;
  s->L_S = p->segment_len;
  s->L_B = p->block_len;
  s->r = s->L_S / s->L_B;
  s->Nq = p->q_len ? (int)p->q_len : s->N;  // chunked prefill: the queries are the last q_len positions
  if (s->Nq > s->N) return EI_ERR_INVALID_ARG;
  s->P = s->N - s->Nq;
  if (s->P % s->L_B) return EI_ERR_UNSUPPORTED_SHAPE;
  s->c0 = s->P / s->L_B;
  s->C_S = (s->Nq + s->L_S - 1) / s->L_S;  // a short last segment / key block when the length is not a multiple
  s->C_B = (s->N + s->L_B - 1) / s->L_B;
  s->SC = ei::row_offset(*s, s->C_S - 1) + ei::causal_blocks(*s, s->C_S - 1);
  s->cells = (int64_t)s->H * s->C_S;
  s->qs_h = p->q_stride_head; s->qs_t = p->q_stride_tok;
  s->ks_h = p->k_stride_head; s->ks_t = p->k_stride_tok;
  s->vs_h = p->v_stride_head; s->vs_t = p->v_stride_tok;
  s->os_h = p->o_stride_head; s->os_t = p->o_stride_tok;
  s->list_div = 1;
  s->KB_cap = s->C_B;
  if ((long double)s->H * s->SC >= 2147483647.0L) return EI_ERR_UNSUPPORTED_SHAPE;  // int32 offsets
  if (s->cells + (int64_t)s->Hkv * s->C_B >= 2147483647LL) return EI_ERR_UNSUPPORTED_SHAPE;
  if (!ei::observe_shape_supported(*s)) return EI_ERR_UNSUPPORTED_SHAPE;
  return EI_OK;
}

template <typename T>
bool dalloc(T** p, size_t n) {
  *p = nullptr;
  return cudaMalloc(reinterpret_cast<void**>(p), n ? n * sizeof(T) : sizeof(T)) == cudaSuccess;
}

struct Item {
  void* ptr;
  size_t bytes;
};
Item item_of(const ei_plan_t* pl, int item) {
  const Shape& s = pl->shape;
  const Shape& ls = pl->lshape;
  switch (item) {
    case EI_ITEM_ENTROPY: return {pl->entropy, sizeof(float) * (size_t)s.cells};
    case EI_ITEM_CLASS: return {pl->rigid, (size_t)ls.H};
    case EI_ITEM_BUDGET: return {pl->kblocks, sizeof(int) * (size_t)ls.cells};
    case EI_ITEM_OFFSETS: return {pl->offsets, sizeof(int) * (size_t)(ls.cells + 1)};
    case EI_ITEM_GROUP_ENTROPY: return {pl->g_entropy, sizeof(float) * (size_t)ls.cells};
    case EI_ITEM_GROUP_SCORES: return {pl->g_scores, sizeof(float) * (size_t)ls.H * (size_t)ls.SC};
    case EI_ITEM_MULTIPLIERS: return {pl->Mfx, sizeof(int) * (size_t)ls.cells};
    case EI_ITEM_INDICES: return {pl->indices, sizeof(int) * (size_t)pl->capacity};
    case EI_ITEM_SCORES: return {pl->scores, sizeof(float) * (size_t)s.H * (size_t)s.SC};
    case EI_ITEM_QMAX: return {pl->qmax, 2 * (size_t)s.cells * s.d};
    case EI_ITEM_QMIN: return {pl->qmin, 2 * (size_t)s.cells * s.d};
    case EI_ITEM_KMAX: return {pl->kmax, 2 * (size_t)s.Hkv * s.KB_cap * s.d};  // head stride KB_cap blocks
    case EI_ITEM_KMIN: return {pl->kmin, 2 * (size_t)s.Hkv * s.KB_cap * s.d};
    case EI_ITEM_STATS: return {pl->stats, sizeof(ei::Stats)};
    default: return {nullptr, 0};
  }
}

}  // namespace

namespace {
// Everything a plan derives from its parameters: the shapes, the configured total, the list capacity it needs.
int derive(ei_plan_t* pl, const ei_params* params, Shape s) {
  if (pl->group) s.list_div = s.G;
  Shape ls = s;
  if (pl->group) {
    ls.H = s.Hkv;
    ls.G = 1;
    ls.cells = (int64_t)s.Hkv * s.C_S;
    ls.list_div = 1;
  }
  const long long lall = (long long)ls.H * ls.SC;
  long long T = 0, b_fx = 0, need = 0;
  if (params->budget_mode == EI_BUDGET_TOTAL_FRACTION) {
    if (!(params->budget_fraction > 0.0) || params->budget_fraction > 1.0) return EI_ERR_INVALID_ARG;
    T = (long long)floor(params->budget_fraction * (double)ls.H * (double)ls.SC + 0.5);
    const int c_last = ei::causal_blocks(ls, ls.C_S - 1);
    const long long forced = (long long)ls.H * ((long long)ls.r * (ls.C_S - 1) + (c_last < ls.r ? c_last : ls.r));  // sum of min(r, C_i)
    if (T < forced || T > lall) return EI_ERR_BUDGET_INFEASIBLE;
    // a plan that holds a shard of a layer's heads can be handed more than its own share of a common total
    need = (params->flags & EI_FLAG_HEAD_SHARD) ? lall : T;
  } else {
    if (!(params->base_budget_tokens > 0.0)) return EI_ERR_INVALID_ARG;
    const double base_blocks = params->base_budget_tokens / (double)s.L_B;
    b_fx = (long long)floor(base_blocks * 4096.0 + 0.5);
    // upper bound sum_i min(C_i, max(r, floor(max_mult * base))) per head
    const long long kcap = (long long)floor(params->max_mult * base_blocks + 1.0);
    long long per_head = 0;
    for (int i = 0; i < s.C_S; ++i) {
      long long Ci = ei::causal_blocks(s, i);
      long long k = kcap < s.r ? s.r : kcap;
      per_head += k < Ci ? k : Ci;
    }
    need = per_head * ls.H;
  }
  pl->shape = s;
  pl->lshape = ls;
  pl->T = T;
  pl->b_fx_base = b_fx;
  pl->need_idx = need;
  pl->obs_scale = params->obs_scale > 0 ? params->obs_scale : 1.0 / sqrt((double)s.d);
  pl->attn_scale = params->attn_scale > 0 ? params->attn_scale : 1.0 / sqrt((double)s.d);
  return EI_OK;
}
}  // namespace

namespace ei {
int shape_from_params(const ei_params* p, Shape* s) { return validate(p, s); }
}  // namespace ei

extern "C" {

int ei_version(void) { return 100; }

const char* ei_status_string(int st) {
  switch (st) {
    case EI_OK: return "ok";
    case EI_ERR_INVALID_ARG: return "invalid argument";
    case EI_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case EI_ERR_BUDGET_INFEASIBLE: return "budget infeasible";
    case EI_ERR_ARCH: return "device is not sm_100";
    case EI_ERR_ALLOC: return "allocation failed";
    case EI_ERR_CUDA: return "CUDA call failed";
    case EI_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case EI_ERR_PLAN_MISMATCH: return "plan mismatch";
    case EI_ERR_NOT_PLANNED: return "plan holds no block lists yet";
    case EI_ERR_SCRATCH_TOO_SMALL: return "shape exceeds the fixed scratch of the allocation-free entry point";
    case EI_ERR_WRONG_DEVICE: return "the current device is not the one the plan was created on";
    default: return "unknown status";
  }
}

int ei_params_default(ei_params* p, int H, int Hkv, int d, int N, int L_S, int L_B, double fraction) {
  if (!p) return EI_ERR_INVALID_ARG;
  memset(p, 0, sizeof(*p));
  p->struct_size = sizeof(ei_params);
  p->n_q_heads = H;
  p->n_kv_heads = Hkv;
  p->head_dim = d;
  p->seq_len = N;
  p->segment_len = L_S;
  p->block_len = L_B;
  p->q_stride_tok = p->k_stride_tok = p->v_stride_tok = p->o_stride_tok = d;
  p->q_stride_head = p->k_stride_head = p->v_stride_head = p->o_stride_head = (int64_t)N * d;
  p->budget_mode = fraction > 0 ? EI_BUDGET_TOTAL_FRACTION : EI_BUDGET_BASE_TOKENS;
  p->budget_fraction = fraction > 0 ? fraction : 0.0;
  p->base_budget_tokens = 2048.0;
  p->entropy_threshold = 1e-5;
  p->alpha = 0.5;
  p->delta_t = 0.4;
  p->max_mult = 3.0;
  p->obs_scale = 0.0;
  p->attn_scale = 0.0;
  p->flags = 0;
  return EI_OK;
}

void ei_plan_destroy(ei_plan_t* pl) {
  if (!pl) return;
  void* ptrs[] = {pl->entropy, pl->rigid, pl->Mfx, pl->kblocks, pl->offsets, pl->indices, pl->scores, pl->qmax,
                  pl->qmin, pl->kmax, pl->kmin, pl->stats, pl->status, pl->sq, pl->sk, pl->sv, pl->so,
                  pl->g_entropy, pl->g_scores, pl->sched, pl->items, pl->pk};
  for (void* p : ptrs)
    if (p) cudaFree(p);
  for (int g = 0; pl->sub && g < pl->shape.Hkv; ++g)
    if (pl->sub[g]) {
      pl->sub[g]->status = nullptr;  // shared with this plan
      ei_plan_destroy(pl->sub[g]);
    }
  delete[] pl->sub;
  if (pl->up) cudaStreamDestroy(pl->up);
  if (pl->down) cudaStreamDestroy(pl->down);
  for (int i = 0; pl->ev && i < pl->n_ev; ++i)
    if (pl->ev[i]) cudaEventDestroy(pl->ev[i]);
  delete[] pl->ev;
  delete pl;
}

int ei_plan_create(const ei_params* params, ei_plan_t** out) {
  if (!out) return EI_ERR_INVALID_ARG;
  *out = nullptr;
  Shape s;
  int rc = validate(params, &s);
  if (rc != EI_OK) return rc;

  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return EI_ERR_CUDA;
  if (prop.major != 10) return EI_ERR_ARCH;

  ei_plan_t* pl = new (std::nothrow) ei_plan_t();
  if (!pl) return EI_ERR_ALLOC;
  memset(pl, 0, sizeof(*pl));
  pl->device = dev;
  pl->params = *params;
  pl->group = (params->flags & EI_FLAG_GROUP_SHARED) != 0;
  rc = derive(pl, params, s);
  if (rc != EI_OK) {
    delete pl;
    return rc;
  }
  s = pl->shape;
  const Shape ls = pl->lshape;
  const long long all = (long long)s.H * s.SC, lall = (long long)ls.H * ls.SC;
  pl->cap_cells = s.cells;
  pl->cap_lcells = ls.cells;
  pl->cap_scores = all;
  pl->cap_lscores = lall;
  pl->capacity = pl->need_idx;

  bool ok = dalloc(&pl->entropy, (size_t)s.cells) && dalloc(&pl->rigid, (size_t)ls.H * ei::MAX_PACKED) &&
            dalloc(&pl->pk, (size_t)ei::MAX_PACKED) &&
            dalloc(&pl->Mfx, (size_t)ls.cells) && dalloc(&pl->kblocks, (size_t)ls.cells) &&
            dalloc(&pl->offsets, (size_t)ls.cells + ei::MAX_PACKED) && dalloc(&pl->indices, (size_t)pl->capacity) &&
            (!pl->group || (dalloc(&pl->g_entropy, (size_t)ls.cells) && dalloc(&pl->g_scores, (size_t)lall))) &&
            dalloc(&pl->scores, (size_t)all) && dalloc(&pl->qmax, (size_t)s.cells * s.d) &&
            dalloc(&pl->qmin, (size_t)s.cells * s.d) && dalloc(&pl->kmax, (size_t)s.Hkv * s.C_B * s.d) &&
            dalloc(&pl->kmin, (size_t)s.Hkv * s.C_B * s.d) && dalloc(&pl->stats, (size_t)ei::MAX_PACKED) && dalloc(&pl->status, 4) &&
            dalloc(&pl->sched, 2) && dalloc(&pl->items, (size_t)ls.cells * (s.L_S >= 256 ? s.L_S / 256 : 1) * 8);
  if (!ok) {
    ei_plan_destroy(pl);
    return EI_ERR_ALLOC;
  }
  if (cudaMemset(pl->status, 0, 4 * sizeof(int)) != cudaSuccess || cudaMemset(pl->sched, 0, 2 * sizeof(int)) != cudaSuccess || cudaMemset(pl->stats, 0, sizeof(ei::Stats)) != cudaSuccess) {
    ei_plan_destroy(pl);
    return EI_ERR_CUDA;
  }
  *out = pl;
  return EI_OK;
}

int ei_stage_pool(ei_plan_t* pl, const void* q, const void* k, void* stream) {
  if (!pl || !q || !k) return EI_ERR_INVALID_ARG;
  if (!on_plan_device(pl)) return EI_ERR_WRONG_DEVICE;
  if (!aligned16(q) || !aligned16(k)) return EI_ERR_UNSUPPORTED_SHAPE;
  cudaError_t e = ei::launch_pool(pl->shape, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, pl->qmax, pl->qmin,
                                  pl->kmax, pl->kmin, pl->k_first, (cudaStream_t)stream);
  pl->launches += 1;
  return e == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

int ei_stage_observe(ei_plan_t* pl, void* stream) {
  if (!pl) return EI_ERR_INVALID_ARG;
  if (!on_plan_device(pl)) return EI_ERR_WRONG_DEVICE;
  cudaError_t e = ei::launch_observe(pl->shape, pl->qmax, pl->qmin, pl->kmax, pl->kmin, pl->obs_scale, pl->scores,
                                     pl->entropy, (cudaStream_t)stream);
  pl->launches += 1;
  if (e == cudaSuccess && pl->group) {
    e = ei::launch_group_aggregate(pl->shape, pl->scores, pl->entropy, pl->g_scores, pl->g_entropy, (cudaStream_t)stream);
    pl->launches += 1;
  }
  return e == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

namespace {
int run_budget(ei_plan_t* pl, int phase, const int* m_all, int n_heads_all, int first_head, long long total_all,
               void* stream) {
  ei::BudgetArgs a;
  a.mode = pl->params.budget_mode;
  a.T = total_all;
  a.b_fx_base = pl->b_fx_base;
  a.e_t = pl->params.entropy_threshold;
  a.alpha = pl->params.alpha;
  a.delta_t = pl->params.delta_t;
  a.max_mult = pl->params.max_mult;
  a.phase = phase;
  a.H_all = n_heads_all;
  a.first_head = first_head;
  cudaError_t e = ei::launch_budget(pl->lshape, a, pl->group ? pl->g_entropy : pl->entropy, pl->rigid, pl->Mfx, m_all,
                                    pl->kblocks, pl->offsets, pl->stats, (cudaStream_t)stream);
  // (with eight heads or more the whole stage is two kernels: the recurrences over several SMs, then the apportionment)
  pl->launches += (phase == ei::EI_BUDGET_PHASE_ALL && pl->lshape.H >= 8) ? 2 : 1;
  return e == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}
}  // namespace

int ei_stage_budget(ei_plan_t* pl, void* stream) {
  if (!pl) return EI_ERR_INVALID_ARG;
  if (!on_plan_device(pl)) return EI_ERR_WRONG_DEVICE;
  return run_budget(pl, ei::EI_BUDGET_PHASE_ALL, nullptr, pl->lshape.H, 0, pl->T, stream);
}

int ei_stage_multipliers(ei_plan_t* pl, int32_t* multipliers_out_dev, void* stream) {
  if (!pl) return EI_ERR_INVALID_ARG;
  if (!on_plan_device(pl)) return EI_ERR_WRONG_DEVICE;
  int rc = run_budget(pl, ei::EI_BUDGET_PHASE_MULTIPLIERS, nullptr, pl->lshape.H, 0, pl->T, stream);
  if (rc == EI_OK && multipliers_out_dev &&
      cudaMemcpyAsync(multipliers_out_dev, pl->Mfx, sizeof(int) * (size_t)pl->lshape.cells, cudaMemcpyDeviceToDevice,
                      (cudaStream_t)stream) != cudaSuccess)
    rc = EI_ERR_CUDA;
  return rc;
}

int ei_stage_apportion(ei_plan_t* pl, const int32_t* multipliers_all_dev, int n_heads_all, int first_head,
                       int64_t total_all, void* stream) {
  if (!pl || !multipliers_all_dev || n_heads_all <= 0 || first_head < 0) return EI_ERR_INVALID_ARG;
  if (!on_plan_device(pl)) return EI_ERR_WRONG_DEVICE;
  const ei::Shape& ls = pl->lshape;
  if (first_head + ls.H > n_heads_all) return EI_ERR_INVALID_ARG;
  if ((long long)n_heads_all * ls.C_S > (1 << 20)) return EI_ERR_UNSUPPORTED_SHAPE;  // one CTA walks every cell
  if (pl->params.budget_mode == EI_BUDGET_TOTAL_FRACTION) {
    const int c_last = ei::causal_blocks(ls, ls.C_S - 1);
    const long long forced1 = (long long)ls.r * (ls.C_S - 1) + (c_last < ls.r ? c_last : ls.r);  // sum of min(r, C_i)
    if (total_all < forced1 * n_heads_all || total_all > (long long)ls.SC * n_heads_all) return EI_ERR_BUDGET_INFEASIBLE;
    // budget flows between the shards: mine may get anything up to all causal blocks of its heads
    const long long all_mine = (long long)ls.H * ls.SC;
    if (pl->capacity < (total_all < all_mine ? total_all : all_mine)) return EI_ERR_PLAN_MISMATCH;
  }
  return run_budget(pl, ei::EI_BUDGET_PHASE_APPORTION, multipliers_all_dev, n_heads_all, first_head, total_all, stream);
}

int ei_stage_select(ei_plan_t* pl, void* stream) {
  if (!pl) return EI_ERR_INVALID_ARG;
  if (!on_plan_device(pl)) return EI_ERR_WRONG_DEVICE;
  const bool quad_shape = pl->shape.L_S % 256 == 0 && pl->shape.d == 128 && pl->shape.L_B == 128;
  cudaError_t e = ei::launch_select(pl->lshape, pl->group ? pl->g_scores : pl->scores, pl->kblocks, pl->offsets,
                                    pl->indices, quad_shape ? pl->items : nullptr, (cudaStream_t)stream);
  pl->launches += 1;
  if (e == cudaSuccess) {
    pl->planned = true;
    pl->items_valid = quad_shape;  // the per-item records of stage 4 follow from the lists alone: made with them
  }
  return e == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

int ei_plan_observe(ei_plan_t* pl, const void* q, const void* k, void* stream) {
  if (!pl || !q || !k) return EI_ERR_INVALID_ARG;
  if (!on_plan_device(pl)) return EI_ERR_WRONG_DEVICE;
  int rc;
  // The fused kernel pays off when every SM gets several rows to pipeline (measured: 6-13 % faster planning at
  // 64k-128k tokens, 10 % slower at 32k where an SM sees fewer than two rows).
  const ei::Shape& s0 = pl->shape;
  const long long rows = (long long)s0.C_S * s0.Hkv;
  const bool want_fused = (pl->params.flags & EI_FLAG_PLAN_FUSED) || rows >= 4 * 148;
  if (ei::pool_observe_shape_supported(pl->shape) && want_fused && !(pl->params.flags & EI_FLAG_PLAN_STAGED)) {
    // K is pooled alone, then one persistent kernel pools the queries and runs the observation behind them
    if (!aligned16(q) || !aligned16(k)) return EI_ERR_UNSUPPORTED_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = ei::launch_pool_k(pl->shape, (const __nv_bfloat16*)k, pl->kmax, pl->kmin, pl->k_first, st);
    if (e == cudaSuccess)
      e = ei::launch_pool_observe(pl->shape, (const __nv_bfloat16*)q, pl->kmax, pl->kmin, pl->qmax, pl->qmin,
                                  pl->obs_scale, pl->scores, pl->entropy, pl->status, st);
    pl->launches += 2;
    if (e == cudaSuccess && pl->group) {
      e = ei::launch_group_aggregate(pl->shape, pl->scores, pl->entropy, pl->g_scores, pl->g_entropy, st);
      pl->launches += 1;
    }
    rc = e == cudaSuccess ? EI_OK : EI_ERR_CUDA;
  } else {
    rc = ei_stage_pool(pl, q, k, stream);
    if (rc == EI_OK) rc = ei_stage_observe(pl, stream);
  }
  return rc;
}

int ei_plan(ei_plan_t* pl, const void* q, const void* k, const void* v, void* stream) {
  (void)v;
  int rc = ei_plan_observe(pl, q, k, stream);
  if (rc == EI_OK) rc = ei_stage_budget(pl, stream);
  if (rc == EI_OK) rc = ei_stage_select(pl, stream);
  return rc;
}

int ei_rope_pool(ei_plan_t* pl, const void* q_in, const void* k_in, const float* cos_table, const float* sin_table,
                 void* q_out, void* k_out, uint32_t flags, void* stream) {
  if (!pl || !q_in || !k_in || !cos_table || !sin_table || !q_out || !k_out || (flags & ~(uint32_t)EI_ROPE_NO_POOL))
    return EI_ERR_INVALID_ARG;
  if (!on_plan_device(pl)) return EI_ERR_WRONG_DEVICE;
  if (!aligned16(q_in) || !aligned16(k_in) || !aligned16(q_out) || !aligned16(k_out) || !aligned16(cos_table) ||
      !aligned16(sin_table))
    return EI_ERR_UNSUPPORTED_SHAPE;
  cudaError_t e = ei::launch_rope_pool(pl->shape, (const __nv_bfloat16*)q_in, (const __nv_bfloat16*)k_in, cos_table,
                                       sin_table, (__nv_bfloat16*)q_out, (__nv_bfloat16*)k_out, pl->qmax, pl->qmin,
                                       pl->kmax, pl->kmin, pl->k_first, !(flags & EI_ROPE_NO_POOL),
                                       (cudaStream_t)stream);
  pl->launches += 1;
  return e == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

int ei_plan_pooled(ei_plan_t* pl, void* stream) {
  if (!pl) return EI_ERR_INVALID_ARG;
  int rc = ei_stage_observe(pl, stream);
  if (rc == EI_OK) rc = ei_stage_budget(pl, stream);
  if (rc == EI_OK) rc = ei_stage_select(pl, stream);
  return rc;
}

// Stage 4 for the query heads of KV heads [g0, g0 + ng): the same kernels on a shape with fewer heads and the
// tensors / list offsets shifted to the first of them.
static int attend(ei_plan_t* pl, const void* q, const void* k, const void* v, void* out, int g0, int ng,
                  cudaStream_t st) {
  const Shape& full = pl->shape;
  Shape s = full;
  s.Hkv = ng;
  s.H = ng * full.G;
  s.cells = (int64_t)s.H * s.C_S;
  const int64_t h0 = (int64_t)g0 * full.G;
  ei::AttnArgs a;
  a.q = (const __nv_bfloat16*)q + h0 * full.qs_h;
  a.k = (const __nv_bfloat16*)k + (int64_t)g0 * full.ks_h;
  a.v = (const __nv_bfloat16*)v + (int64_t)g0 * full.vs_h;
  a.out = (__nv_bfloat16*)out + h0 * full.os_h;
  a.offsets = pl->offsets + (h0 / full.list_div) * full.C_S;  // the entries are positions in the whole index array
  a.indices = pl->indices;
  a.status = pl->status;
  a.scale = (float)pl->attn_scale;
  a.p_via_smem = (pl->params.flags & EI_FLAG_ATTN_P_VIA_SMEM) != 0;
  a.single_tile = (pl->params.flags & EI_FLAG_ATTN_SINGLE_TILE) != 0;
  a.pair_8warp = (pl->params.flags & EI_FLAG_ATTN_PAIR_8WARP) != 0;
  a.persistent = (pl->params.flags & EI_FLAG_ATTN_PERSISTENT) != 0;
  // head_dim 128, 128-wide blocks, segments a multiple of 256: the quad-layout kernel, one CTA per tile pair, unless
  // a flag asks for another kernel (the split-row kernels are the only ones that can leave out all-zero P.V products)
  const bool quad_shape = full.L_S % 256 == 0 && full.d == 128 && full.L_B == 128;
  const uint32_t other = EI_FLAG_ATTN_SPLIT | EI_FLAG_ATTN_SKIP_ZERO_PV | EI_FLAG_ATTN_P_VIA_SMEM | EI_FLAG_ATTN_PAIR_8WARP;
  a.quad_kernel = quad_shape && !(pl->params.flags & other) &&
                  ((pl->params.flags & EI_FLAG_ATTN_QUAD) ||
                   !(pl->params.flags & (EI_FLAG_ATTN_PERSISTENT | EI_FLAG_ATTN_SINGLE_TILE)));
  a.tri_kernel = quad_shape && (pl->params.flags & EI_FLAG_ATTN_TRI) != 0;
  a.tri_tiles = 0;
  if (a.tri_kernel) a.quad_kernel = false;
  a.items = nullptr;
  if (a.quad_kernel || a.tri_kernel) {
    if (!pl->items_valid) {  // the lists changed since the records were made
      if (ei::launch_attention_items(pl->lshape, pl->offsets, pl->indices, pl->items, st) != cudaSuccess) return EI_ERR_CUDA;
      pl->items_valid = true;
      pl->launches += 1;
    }
    a.items = pl->items + (h0 / full.list_div) * full.C_S * (full.L_S / 256) * 8;
  }
  a.sched = pl->sched;
  a.skip_log2 = (pl->params.flags & EI_FLAG_ATTN_NO_SKIP) ? INFINITY : 24.0f;
  a.pv_skipped = (pl->params.flags & EI_FLAG_ATTN_SKIP_ZERO_PV) ? &pl->stats->pv_skipped : nullptr;
  const int rc = ei::launch_attention(s, a, st);
  pl->launches += 1;
  return rc;
}

int ei_sparse_prefill(const ei_plan_t* pl, const void* q, const void* k, const void* v, void* out, void* stream) {
  if (!pl || !q || !k || !v || !out) return EI_ERR_INVALID_ARG;
  if (!on_plan_device(pl)) return EI_ERR_WRONG_DEVICE;
  if (!pl->planned) return EI_ERR_NOT_PLANNED;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return EI_ERR_UNSUPPORTED_SHAPE;
  return attend(const_cast<ei_plan_t*>(pl), q, k, v, out, 0, pl->shape.Hkv, (cudaStream_t)stream);
}

// Host path.  The copies run on two streams of the plan's own so that PCIe carries both directions at once:
//   upload stream:   K, Q, then V one KV head at a time
//   caller's stream: ei_plan once K and Q are there (in TOTAL mode the budgets couple all heads, so nothing can
//                    be attended before every head's entropy is known), then stage 4 one KV group at a time as
//                    its V arrives
//   download stream: each group's output as soon as it is written, under the remaining V uploads and groups
int ei_prefill_host(ei_plan_t* pl, const void* qh, const void* kh, const void* vh, void* oh, void* stream) {
  if (!pl || !qh || !kh || !vh || !oh) return EI_ERR_INVALID_ARG;
  if (!on_plan_device(pl)) return EI_ERR_WRONG_DEVICE;
  const Shape& s = pl->shape;
  const ei_params& p = pl->params;
  if (p.q_stride_tok != s.d || p.k_stride_tok != s.d || p.v_stride_tok != s.d || p.o_stride_tok != s.d ||
      p.q_stride_head != (int64_t)s.Nq * s.d || p.k_stride_head != (int64_t)s.N * s.d ||
      p.v_stride_head != (int64_t)s.N * s.d || p.o_stride_head != (int64_t)s.Nq * s.d)
    return EI_ERR_UNSUPPORTED_SHAPE;  // the host path is for contiguous tensors
  const size_t nq = (size_t)s.H * s.Nq * s.d, nk = (size_t)s.Hkv * s.N * s.d;
  if (nq > pl->stage_nq || nk > pl->stage_nk) {  // first use, or the plan was re-targeted to a longer problem since
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return EI_ERR_CUDA;
    for (__nv_bfloat16** b : {&pl->sq, &pl->sk, &pl->sv, &pl->so}) {
      if (*b) cudaFree(*b);
      *b = nullptr;
    }
    pl->stage_nq = pl->stage_nk = 0;
    if (!dalloc(&pl->sq, nq) || !dalloc(&pl->sk, nk) || !dalloc(&pl->sv, nk) || !dalloc(&pl->so, nq)) return EI_ERR_ALLOC;
    pl->stage_nq = nq;
    pl->stage_nk = nk;
  }
  if (!pl->up) {
    if (cudaStreamCreateWithFlags(&pl->up, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&pl->down, cudaStreamNonBlocking) != cudaSuccess)
      return EI_ERR_CUDA;
    pl->n_ev = 3 + 2 * s.Hkv;
    pl->ev = new (std::nothrow) cudaEvent_t[pl->n_ev]();
    if (!pl->ev) return EI_ERR_ALLOC;
    for (int i = 0; i < pl->n_ev; ++i)
      if (cudaEventCreateWithFlags(&pl->ev[i], cudaEventDisableTiming) != cudaSuccess) return EI_ERR_CUDA;
  }
  if (pl->n_ev < 3 + 2 * s.Hkv) return EI_ERR_PLAN_MISMATCH;
  cudaStream_t st = (cudaStream_t)stream;
  cudaEvent_t ev_in = pl->ev[0], ev_kq = pl->ev[1], ev_done = pl->ev[2];
  cudaEvent_t* ev_v = pl->ev + 3;
  cudaEvent_t* ev_a = pl->ev + 3 + s.Hkv;
  bool ok = cudaEventRecord(ev_in, st) == cudaSuccess &&  // work already queued by the caller comes first
            cudaStreamWaitEvent(pl->up, ev_in, 0) == cudaSuccess &&
            cudaStreamWaitEvent(pl->down, ev_in, 0) == cudaSuccess;
  const size_t k_head = (size_t)s.N * s.d, v_head = k_head, o_group = (size_t)s.G * s.Nq * s.d;
  int rc = EI_OK;
  if (p.budget_mode == EI_BUDGET_BASE_TOKENS && s.Hkv > 1) {
    // BASE mode: the budgets of a head depend on that head alone, so every KV group is a problem of its own --
    // upload its K, V and Q, plan and attend it (in a plan of its own), send its output back, all while the next
    // groups are still on their way up.  The plan's own tables are not filled by this form of the call.
    if (!pl->sub) {
      pl->sub = new (std::nothrow) ei_plan_s*[s.Hkv]();
      if (!pl->sub) return EI_ERR_ALLOC;
    }
    ei_params sp = p;
    sp.n_q_heads = s.G;
    sp.n_kv_heads = 1;
    for (int g = 0; g < s.Hkv; ++g) {
      if (pl->sub[g] && ei_plan_set_lengths(pl->sub[g], p.seq_len, (int)p.q_len, 0) != EI_OK) {
        pl->sub[g]->status = nullptr;  // made for a shorter problem: replace it
        ei_plan_destroy(pl->sub[g]);
        pl->sub[g] = nullptr;
      }
      if (!pl->sub[g]) {
        const int crc = ei_plan_create(&sp, &pl->sub[g]);
        if (crc != EI_OK) return crc;
        cudaFree(pl->sub[g]->status);
        pl->sub[g]->status = pl->status;  // one status word for the whole call
      }
    }
    for (int g = 0; ok && g < s.Hkv; ++g)
      ok = cudaMemcpyAsync(pl->sk + g * k_head, (const __nv_bfloat16*)kh + g * k_head, k_head * 2,
                           cudaMemcpyHostToDevice, pl->up) == cudaSuccess &&
           cudaMemcpyAsync(pl->sq + g * o_group, (const __nv_bfloat16*)qh + g * o_group, o_group * 2,
                           cudaMemcpyHostToDevice, pl->up) == cudaSuccess &&
           cudaMemcpyAsync(pl->sv + g * v_head, (const __nv_bfloat16*)vh + g * v_head, v_head * 2,
                           cudaMemcpyHostToDevice, pl->up) == cudaSuccess &&
           cudaEventRecord(ev_v[g], pl->up) == cudaSuccess;
    if (!ok) rc = EI_ERR_CUDA;  // (falls through to the join below: copies already queued must not outlive the call)
    for (int g = 0; rc == EI_OK && g < s.Hkv; ++g) {
      ei_plan_t* sb = pl->sub[g];
      const __nv_bfloat16 *qg = pl->sq + g * o_group, *kg = pl->sk + g * k_head, *vg = pl->sv + g * v_head;
      const long long l0 = sb->launches;
      if (cudaStreamWaitEvent(st, ev_v[g], 0) != cudaSuccess) rc = EI_ERR_CUDA;
      if (rc == EI_OK) rc = ei_plan(sb, qg, kg, vg, stream);
      if (rc == EI_OK) rc = ei_sparse_prefill(sb, qg, kg, vg, pl->so + g * o_group, stream);
      pl->launches += sb->launches - l0;
      if (rc == EI_OK && (cudaEventRecord(ev_a[g], st) != cudaSuccess ||
                          cudaStreamWaitEvent(pl->down, ev_a[g], 0) != cudaSuccess ||
                          cudaMemcpyAsync((__nv_bfloat16*)oh + g * o_group, pl->so + g * o_group, o_group * 2,
                                          cudaMemcpyDeviceToHost, pl->down) != cudaSuccess))
        rc = EI_ERR_CUDA;
    }
  } else {
    ok = ok && cudaMemcpyAsync(pl->sk, kh, nk * 2, cudaMemcpyHostToDevice, pl->up) == cudaSuccess &&
         cudaMemcpyAsync(pl->sq, qh, nq * 2, cudaMemcpyHostToDevice, pl->up) == cudaSuccess &&
         cudaEventRecord(ev_kq, pl->up) == cudaSuccess;
    for (int g = 0; ok && g < s.Hkv; ++g)
      ok = cudaMemcpyAsync(pl->sv + g * v_head, (const __nv_bfloat16*)vh + g * v_head, v_head * 2, cudaMemcpyHostToDevice,
                           pl->up) == cudaSuccess &&
           cudaEventRecord(ev_v[g], pl->up) == cudaSuccess;
    if (!ok || cudaStreamWaitEvent(st, ev_kq, 0) != cudaSuccess) rc = EI_ERR_CUDA;  // (joined below all the same)
    if (rc == EI_OK) rc = ei_plan(pl, pl->sq, pl->sk, pl->sv, stream);
    for (int g = 0; rc == EI_OK && g < s.Hkv; ++g) {
      if (cudaStreamWaitEvent(st, ev_v[g], 0) != cudaSuccess) rc = EI_ERR_CUDA;
      if (rc == EI_OK) rc = attend(pl, pl->sq, pl->sk, pl->sv, pl->so, g, 1, st);
      if (rc == EI_OK && (cudaEventRecord(ev_a[g], st) != cudaSuccess ||
                          cudaStreamWaitEvent(pl->down, ev_a[g], 0) != cudaSuccess ||
                          cudaMemcpyAsync((__nv_bfloat16*)oh + g * o_group, pl->so + g * o_group, o_group * 2,
                                          cudaMemcpyDeviceToHost, pl->down) != cudaSuccess))
        rc = EI_ERR_CUDA;
    }
  }
  // whatever happened, leave nothing of this call in flight on the plan's streams
  const bool joined = cudaEventRecord(ev_done, pl->down) == cudaSuccess &&
                      cudaStreamWaitEvent(st, ev_done, 0) == cudaSuccess &&
                      cudaStreamSynchronize(pl->up) == cudaSuccess && cudaStreamSynchronize(st) == cudaSuccess;
  if (rc != EI_OK) return rc;
  return joined ? EI_OK : EI_ERR_CUDA;
}

int ei_plan_debug_waits(ei_plan_t* pl, int wait_limit_log2, int skip_ring_item, void* stream) {
  if (!pl || wait_limit_log2 < 0 || wait_limit_log2 >= 40 || skip_ring_item < -1) return EI_ERR_INVALID_ARG;
  if (!on_plan_device(pl)) return EI_ERR_WRONG_DEVICE;
  const int v[2] = {wait_limit_log2, skip_ring_item + 1};
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(pl->status + 1, v, sizeof(v), cudaMemcpyHostToDevice, st) != cudaSuccess) return EI_ERR_CUDA;
  return cudaStreamSynchronize(st) == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

int ei_plan_get(const ei_plan_t* pl, int item, const void** dev_ptr, size_t* bytes) {
  if (!pl) return EI_ERR_INVALID_ARG;
  Item it = item_of(pl, item);
  if (!it.ptr) return EI_ERR_INVALID_ARG;
  if (dev_ptr) *dev_ptr = it.ptr;
  if (bytes) *bytes = it.bytes;
  return EI_OK;
}

int ei_plan_read(const ei_plan_t* pl, int item, void* host_dst, size_t bytes, void* stream) {
  if (!pl || !host_dst) return EI_ERR_INVALID_ARG;
  Item it = item_of(pl, item);
  if (!it.ptr || bytes > it.bytes) return EI_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(host_dst, it.ptr, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return EI_ERR_CUDA;
  return cudaStreamSynchronize(st) == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

int ei_plan_write(ei_plan_t* pl, int item, const void* host_src, size_t bytes, void* stream) {
  if (!pl || !host_src) return EI_ERR_INVALID_ARG;
  Item it = item_of(pl, item);
  if (!it.ptr || bytes > it.bytes) return EI_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(it.ptr, host_src, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return EI_ERR_CUDA;
  pl->items_valid = false;  // the item may be part of the lists
  return cudaStreamSynchronize(st) == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

int ei_plan_set_lists(ei_plan_t* pl, const int32_t* k_host, const int32_t* idx_host, size_t n_idx, void* stream) {
  if (!pl || !k_host || (!idx_host && n_idx)) return EI_ERR_INVALID_ARG;
  const Shape& s = pl->lshape;
  if ((long long)n_idx > pl->capacity) return EI_ERR_PLAN_MISMATCH;
  std::vector<int> off((size_t)s.cells + 1);
  long long run = 0;
  for (long long c = 0; c < s.cells; ++c) {
    off[(size_t)c] = (int)run;
    const int kc = k_host[c];
    const int Ci = ei::causal_blocks(s, (int)(c % s.C_S));
    if (kc < 0 || kc > Ci || run + kc > (long long)n_idx) return EI_ERR_PLAN_MISMATCH;
    for (int t = 0; t < kc; ++t) {
      const int j = idx_host[run + t];
      if (j < 0 || j >= Ci || (t > 0 && j <= idx_host[run + t - 1])) return EI_ERR_PLAN_MISMATCH;
    }
    run += kc;
  }
  off[(size_t)s.cells] = (int)run;
  if (run != (long long)n_idx) return EI_ERR_PLAN_MISMATCH;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(pl->kblocks, k_host, sizeof(int) * (size_t)s.cells, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(pl->offsets, off.data(), sizeof(int) * off.size(), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      (n_idx && cudaMemcpyAsync(pl->indices, idx_host, sizeof(int) * n_idx, cudaMemcpyHostToDevice, st) != cudaSuccess))
    return EI_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return EI_ERR_CUDA;
  pl->planned = true;
  pl->items_valid = false;
  return EI_OK;
}

int ei_plan_set_lengths(ei_plan_t* pl, int seq_len, int q_len, int k_blocks_valid) {
  if (!pl || seq_len <= 0 || q_len < 0 || k_blocks_valid < 0) return EI_ERR_INVALID_ARG;
  ei_params p = pl->params;
  p.seq_len = seq_len;
  p.q_len = (uint32_t)q_len;
  Shape s;
  int rc = validate(&p, &s);
  if (rc != EI_OK) return rc;
  const int kb_cap = pl->shape.KB_cap;
  if (s.C_B > kb_cap || k_blocks_valid > s.C_B) return EI_ERR_PLAN_MISMATCH;
  s.KB_cap = kb_cap;
  ei_plan_t probe = *pl;  // derive into a copy first: the plan stays as it is when the new shape does not fit
  rc = derive(&probe, &p, s);
  if (rc != EI_OK) return rc;
  const Shape &ns = probe.shape, &nl = probe.lshape;
  if (ns.cells > pl->cap_cells || nl.cells > pl->cap_lcells || (long long)ns.H * ns.SC > pl->cap_scores ||
      (long long)nl.H * nl.SC > pl->cap_lscores || probe.need_idx > pl->capacity)
    return EI_ERR_PLAN_MISMATCH;
  probe.params = p;
  probe.k_first = k_blocks_valid;
  probe.planned = false;
  probe.items_valid = false;
  *pl = probe;
  return EI_OK;
}

namespace {
// Can a packed batch run in one set of launches on this plan?  (The staged planning kernels and the stage-4
// kernels picked by default take the per-sequence table; the kernels behind flags go sequence by sequence.)
bool packed_capable(const ei_plan_t* pl) {
  const uint32_t other = EI_FLAG_ATTN_SPLIT | EI_FLAG_ATTN_SKIP_ZERO_PV | EI_FLAG_ATTN_P_VIA_SMEM |
                         EI_FLAG_ATTN_PAIR_8WARP | EI_FLAG_ATTN_PERSISTENT | EI_FLAG_ATTN_SINGLE_TILE | EI_FLAG_ATTN_TRI |
                         EI_FLAG_ATTN_QUAD;
  return !(pl->params.flags & other);
}

// sequences [b0, b1) of the batch (all non-empty, all fitting the plan's tables together) in five launches
int run_packed(ei_plan_t* pl, const std::vector<ei::PackedSeq>& seqs_in, long long n_tokens, const void* q, const void* k,
               const void* v, void* out, cudaStream_t st) {
  std::vector<ei::PackedSeq> hp(seqs_in);
  const int n = (int)hp.size();
  ei::packed_fill_work(hp.data(), n);
  if (cudaMemcpyAsync(pl->pk, hp.data(), sizeof(ei::PackedSeq) * n, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return EI_ERR_CUDA;
  cudaError_t e = ei::launch_pool_packed(pl->pk, hp.data(), n, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, pl->qmax,
                                         pl->qmin, pl->kmax, pl->kmin, st);
  if (e == cudaSuccess)
    e = ei::launch_observe_packed(pl->pk, hp.data(), n, pl->qmax, pl->qmin, pl->kmax, pl->kmin, pl->obs_scale, pl->scores,
                                  pl->entropy, st);
  ei::BudgetArgs a;
  a.mode = pl->params.budget_mode;
  a.T = 0;
  a.b_fx_base = pl->b_fx_base;
  a.e_t = pl->params.entropy_threshold;
  a.alpha = pl->params.alpha;
  a.delta_t = pl->params.delta_t;
  a.max_mult = pl->params.max_mult;
  a.phase = ei::EI_BUDGET_PHASE_ALL;
  a.H_all = 0;
  a.first_head = 0;
  if (e == cudaSuccess && pl->group) {
    e = ei::launch_group_aggregate_packed(pl->pk, hp.data(), n, pl->scores, pl->entropy, pl->g_scores, pl->g_entropy, st);
    pl->launches += 1;
  }
  if (e == cudaSuccess)
    e = ei::launch_budget_packed(pl->pk, n, a, pl->group ? pl->g_entropy : pl->entropy, pl->rigid, pl->Mfx, pl->kblocks,
                                 pl->offsets, pl->stats, st);
  if (e == cudaSuccess)
    e = ei::launch_select_packed(pl->pk, hp.data(), n, pl->group ? pl->g_scores : pl->scores, pl->kblocks, pl->offsets,
                                 pl->indices, pl->items, st);
  pl->launches += 4;
  if (e != cudaSuccess) return EI_ERR_CUDA;
  ei::AttnArgs at{};
  at.q = (const __nv_bfloat16*)q;
  at.k = (const __nv_bfloat16*)k;
  at.v = (const __nv_bfloat16*)v;
  at.out = (__nv_bfloat16*)out;
  at.offsets = pl->offsets;
  at.indices = pl->indices;
  at.items = pl->items;
  at.status = pl->status;
  at.scale = (float)pl->attn_scale;
  at.skip_log2 = (pl->params.flags & EI_FLAG_ATTN_NO_SKIP) ? INFINITY : 24.0f;
  const int rc = ei::launch_attention_packed(pl->pk, hp.data(), n, n_tokens, at, st);
  pl->launches += 1;
  return rc;
}
}  // namespace

int ei_prefill_varlen(ei_plan_t* pl, const void* q, const void* k, const void* v, void* out,
                      const int32_t* cu_seqlens_host, int n_seqs, void* stream) {
  if (!pl || !q || !k || !v || !out || !cu_seqlens_host || n_seqs < 0) return EI_ERR_INVALID_ARG;
  if (pl->params.q_len != 0 && (int)pl->params.q_len != pl->params.seq_len) return EI_ERR_INVALID_ARG;  // whole prefills only
  const int32_t* cu = cu_seqlens_host;
  if (cu[0] < 0) return EI_ERR_INVALID_ARG;
  for (int b = 0; b < n_seqs; ++b)
    if (cu[b + 1] < cu[b]) return EI_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return EI_ERR_UNSUPPORTED_SHAPE;
  // every sequence has to fit the plan before anything is launched (host-only probes); what a plan of each
  // sequence alone would look like is kept for the packed launches
  const ei_plan_t saved = *pl;
  std::vector<ei::PackedSeq> seqs;
  std::vector<long long> need;
  for (int b = 0; b < n_seqs; ++b) {
    const int len = cu[b + 1] - cu[b];
    if (len == 0) continue;
    const int rc = ei_plan_set_lengths(pl, len, 0, 0);
    if (rc != EI_OK) {
      *pl = saved;
      return rc;
    }
    ei::PackedSeq P{};
    P.s = pl->shape;
    P.s.KB_cap = P.s.C_B;  // its K representatives are laid out as a plan of this sequence alone would lay them out
    P.ls = pl->lshape;
    P.ls.KB_cap = P.ls.C_B;
    P.tok0 = cu[b];
    P.T = pl->T;
    P.index = b;  // (the batch position for now; the slot within its set of launches is assigned below)
    seqs.push_back(P);
    need.push_back(pl->need_idx);
  }
  const ei_params& p = pl->params;
  const bool packed_ok = packed_capable(pl) && ei::observe_shape_supported(pl->shape);
  const long long n_tokens = cu[n_seqs];
  const long long kreps_cap = (long long)saved.shape.Hkv * saved.shape.KB_cap;
  cudaStream_t st = (cudaStream_t)stream;
  size_t i0 = 0;
  bool last_packed = false;
  while (i0 < seqs.size()) {
    // the longest run of sequences from i0 on whose tables fit the plan's side by side
    size_t i1 = i0;
    long long cells = 0, sc = 0, kb = 0, idx = 0, lcells = 0, lsc = 0;
    std::vector<ei::PackedSeq> grp;
    while (packed_ok && i1 < seqs.size() && (int)grp.size() < ei::MAX_PACKED) {
      const ei::Shape &sb = seqs[i1].s, &lb = seqs[i1].ls;
      if (cells + sb.cells > pl->cap_cells || sc + (long long)sb.H * sb.SC > pl->cap_scores ||
          lcells + lb.cells > pl->cap_lcells || lsc + (long long)lb.H * lb.SC > pl->cap_lscores ||
          kb + (long long)sb.Hkv * sb.C_B > kreps_cap || idx + need[i1] > pl->capacity)
        break;
      ei::PackedSeq P = seqs[i1];
      P.cell0 = cells;
      P.lcell0 = lcells;
      P.off0 = lcells + (long long)grp.size();
      P.sc0 = sc;
      P.lsc0 = lsc;
      P.kb0 = kb;
      P.idx0 = idx;
      P.head0 = (int)grp.size() * lb.H;
      P.index = (int)grp.size();
      grp.push_back(P);
      cells += sb.cells;
      lcells += lb.cells;
      lsc += (long long)lb.H * lb.SC;
      sc += (long long)sb.H * sb.SC;
      kb += (long long)sb.Hkv * sb.C_B;
      idx += need[i1];
      ++i1;
    }
    int rc;
    if (grp.size() >= 2) {
      rc = run_packed(pl, grp, n_tokens, q, k, v, out, st);
      last_packed = true;
    } else {  // one sequence on its own: the plan re-targeted to it, the ordinary two calls
      i1 = i0 + 1;
      const long long t0 = seqs[i0].tok0;
      rc = ei_plan_set_lengths(pl, seqs[i0].s.N, 0, 0);
      const __nv_bfloat16* qb = (const __nv_bfloat16*)q + t0 * p.q_stride_tok;
      const __nv_bfloat16* kb1 = (const __nv_bfloat16*)k + t0 * p.k_stride_tok;
      const __nv_bfloat16* vb = (const __nv_bfloat16*)v + t0 * p.v_stride_tok;
      __nv_bfloat16* ob = (__nv_bfloat16*)out + t0 * p.o_stride_tok;
      if (rc == EI_OK) rc = ei_plan(pl, qb, kb1, vb, stream);
      if (rc == EI_OK) rc = ei_sparse_prefill(pl, qb, kb1, vb, ob, stream);
      last_packed = false;
    }
    if (rc != EI_OK) return rc;
    i0 = i1;
  }
  if (!seqs.empty()) {
    ei_plan_set_lengths(pl, seqs.back().s.N, 0, 0);  // left targeted at the last non-empty sequence
    if (last_packed) {  // the tables hold a batch, not that sequence: nothing to attend from until the next ei_plan
      pl->planned = false;
      pl->items_valid = false;
    }
  }
  return EI_OK;
}

int ei_plan_status(ei_plan_t* pl, void* stream) {
  if (!pl) return EI_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int v = 0;
  if (cudaMemcpyAsync(&v, pl->status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return EI_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return EI_ERR_CUDA;
  if (v != 0) {
    if (cudaMemsetAsync(pl->status, 0, sizeof(int), st) != cudaSuccess) return EI_ERR_CUDA;
    cudaStreamSynchronize(st);
  }
  return v;
}

int64_t ei_plan_total_blocks(const ei_plan_t* pl) {
  if (!pl) return -1;
  return pl->params.budget_mode == EI_BUDGET_TOTAL_FRACTION ? pl->T : pl->capacity;
}

int64_t ei_plan_launches(const ei_plan_t* pl) { return pl ? pl->launches : -1; }

}  // extern "C"
