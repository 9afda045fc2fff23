// Latent KV-cache compression (appendix "Latent KV Cache Compression Algorithm", Algorithm 4; Section 4.3),
// sm_100a.  Per KV head g, with the G query heads of its group and an observation window of N_W query rows:
//   w_j = sum_i (Q_W K^T)[i, j]                         raw logits, as printed
//   keep the B_d positions with the largest w (ties: lower position), in increasing position order
//   K_out[t] = K[idx[t]],  V_out[t] = V[idx[t]]
// Because the column sums of Q_W K^T are (sum_i q_i) . k_j, the scoring is one pass over K:
//   qsum_kernel    qsum[g,:] = sum over the group's heads and the window rows of q            (tiny)
//   score_kernel   w[g,j] = qsum[g,:] . K[g,j,:]    HBM-bound, 16-byte loads, half a warp per key row;
//                  also counts the top 12 bits of the order-preserving score keys per KV head
//   topk_kernel    per KV head (one CTA): threshold key of rank B_d from that histogram plus three light
//                  radix passes, then an index-ordered compaction (equal keys: the lowest positions)
//   gather_kernel  copies the kept K and V rows                                                 HBM-bound
#include <cooperative_groups.h>
#include "ei_internal.cuh"

namespace ei {

namespace {

constexpr int CMP_THREADS = 256;
constexpr int TOPK_THREADS = 1024;
constexpr int HIST12 = 4096;
#ifndef SCORE_CTAS_PER_SM
#define SCORE_CTAS_PER_SM 2  // resident CTAs of the scoring pass per SM (98 registers x 256 threads)
#endif
#ifndef SCORE_TILES
#define SCORE_TILES 1  // 16-row tiles per warp step of the scoring pass at d = 128 (twice that at d = 64)
#endif

// Programmatic dependent launch: the four kernels of a call form a chain; each lets its successor start early
// (its CTAs take SMs as they fall free and run their own set-up) and waits, before it touches anything the
// chain produces, until its predecessor has finished and its writes are visible.  Pointers to data the chain
// produces carry no __restrict__ in the consumer: a load known to be read-only may be moved above the wait.
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ uint32_t order_key_f(float f) {
  f += 0.0f;  // -0 -> +0
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// qsum[g, c] = sum_{h in group g} sum_{i < N_W} q[h, i, c]: one CTA per KV head; a thread adds every
// (256/LPR)-th window row of its 16-byte column in fp32, then the row slots are added in a fixed order.
template <int D>
__global__ void __launch_bounds__(CMP_THREADS) qsum_kernel(const __nv_bfloat16* __restrict__ qw, float* __restrict__ qsum,
                                                           int* __restrict__ hist12, int G, int N_W, long long qs_h,
                                                           long long qs_t) {
  constexpr int LPR = D / 8, RS = CMP_THREADS / LPR;
  __shared__ float part[RS][D];
  const int g = blockIdx.x, lane16 = threadIdx.x % LPR, slot = threadIdx.x / LPR;
  chain_release();
  for (int b = threadIdx.x; b < HIST12; b += CMP_THREADS) hist12[g * HIST12 + b] = 0;  // the scoring pass adds into it
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int r0 = slot; r0 < G * N_W; r0 += RS * 8) {  // eight loads in flight; the adds keep the row order
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int r = r0 + u * RS;
      if (r < G * N_W) v[u] = *reinterpret_cast<const uint4*>(qw + (r / N_W + g * G) * qs_h + (r % N_W) * qs_t + lane16 * 8);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (r0 + u * RS >= G * N_W) break;
      const uint32_t ws[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        acc[2 * e] += __uint_as_float(ws[e] << 16);
        acc[2 * e + 1] += __uint_as_float(ws[e] & 0xFFFF0000u);
      }
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) part[slot][lane16 * 8 + e] = acc[e];
  __syncthreads();
  if (threadIdx.x < D) {
    float t = 0.f;
    for (int r = 0; r < RS; ++r) t += part[r][threadIdx.x];
    qsum[(long long)g * D + threadIdx.x] = t;
  }
}

// w[g, j] = qsum[g, :] . K[g, j, :] for 16 rows per warp step on the bf16 tensor-core path (mma.m16n8k16, fp32
// accumulate), used here only to keep the instruction count of an HBM-bound pass low.  qsum is split into three
// bf16 terms (hi + mid + lo carries all 24 bits of the fp32 value) that sit in columns 0..2 of the B operand;
// the bf16 x bf16 products are exact and the three column sums are added at the end.  A dot product does not
// care in which order the d index is walked, so each lane feeds the 16 bytes it loaded straight into the A
// fragment and B is laid out to match: lane (g = lane / 4, t = lane % 4) loads bytes [128 n + 32 t, +32) of rows
// g and g + 8 for each 128-byte line n of the row, so every load instruction of a warp covers whole lines.
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// term `part` (0 hi, 1 mid, 2 lo, else zero) of the three-way bf16 split of x, as bf16 bits
__device__ __forceinline__ uint32_t bf16_split_term(float x, int part) {
  if (part > 2) return 0u;
  __nv_bfloat16 h = __float2bfloat16_rn(x);
  for (int i = 0; i < part; ++i) {
    x -= __bfloat162float(h);  // exact: the remainder of a bf16 rounding fits fp32
    h = __float2bfloat16_rn(x);
  }
  return (uint32_t)__bfloat16_as_ushort(h);
}

struct u32x8 {
  uint32_t r[8];
};
// one 32-byte streaming load (the 256-bit global load of sm_100)
__device__ __forceinline__ u32x8 ld_stream_32B(const void* p) {
  u32x8 v;
  asm volatile("ld.global.cs.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(v.r[0]), "=r"(v.r[1]), "=r"(v.r[2]), "=r"(v.r[3]), "=r"(v.r[4]), "=r"(v.r[5]), "=r"(v.r[6]),
                 "=r"(v.r[7])
               : "l"(p));
  return v;
}

// WIDE: the rows are 32-byte aligned and one 256-bit load fetches a lane's share; otherwise two 16-byte loads do
template <int D, bool WIDE>
__global__ void __launch_bounds__(CMP_THREADS) score_kernel(const __nv_bfloat16* __restrict__ k,
                                                            const float* qsum, float* __restrict__ w,
                                                            int* __restrict__ hist12, int L, int Hkv,
                                                            long long ks_h, long long ks_t) {
  constexpr int NLINE = D / 64;                 // 128-byte lines per row; a quad of lanes loads one line of a row
  constexpr int T = SCORE_TILES * 128 / D > 0 ? SCORE_TILES * 128 / D : 1;  // 16-row tiles a warp has in flight
  constexpr int ROWS_PER_CTA = (CMP_THREADS / 32) * 16 * T;
  __shared__ int sh[HIST12];  // this CTA's counts of the top 12 bits of the order-preserving score keys
  chain_release();
  for (int b = threadIdx.x; b < HIST12; b += CMP_THREADS) sh[b] = 0;
  __syncthreads();
  chain_wait();  // qsum and the zeroed global histogram come from the kernel before
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, grp = lane >> 2, t4 = lane & 3;
  // The CTAs of grid row y stay on head y and walk its tiles of 16 * T rows per warp with stride gridDim.x.  Two
  // tile buffers leapfrog: while one tile is multiplied, the loads of the next are in flight.
  const int g = blockIdx.y;
  const int n_tiles = (L + ROWS_PER_CTA - 1) / ROWS_PER_CTA;
  uint32_t bq[NLINE][4][2];
#pragma unroll
  for (int ln = 0; ln < NLINE; ++ln)
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      const float* qp = qsum + (long long)g * D + 64 * ln + 16 * t4 + 4 * m;
      bq[ln][m][0] = bf16_split_term(qp[0], grp) | (bf16_split_term(qp[1], grp) << 16);
      bq[ln][m][1] = bf16_split_term(qp[2], grp) | (bf16_split_term(qp[3], grp) << 16);
    }
  const __nv_bfloat16* base = k + (long long)g * ks_h + t4 * 16;
  float* wg = w + (long long)g * L;
  auto load_tile = [&](u32x8 (&v)[T][2][NLINE], int ptile) {
    const long long r0 = (long long)ptile * ROWS_PER_CTA + warp * 16 * T;
#pragma unroll
    for (int tt = 0; tt < T; ++tt)
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const long long row = r0 + tt * 16 + hh * 8 + grp;
        const __nv_bfloat16* rp = base + row * ks_t;
#pragma unroll
        for (int ln = 0; ln < NLINE; ++ln) {
          if (ptile < n_tiles && row < L) {
            if (WIDE) {
              v[tt][hh][ln] = ld_stream_32B(rp + ln * 64);
            } else {
              const uint4 x = __ldcs(reinterpret_cast<const uint4*>(rp + ln * 64));
              const uint4 y = __ldcs(reinterpret_cast<const uint4*>(rp + ln * 64 + 8));
              v[tt][hh][ln] = u32x8{{x.x, x.y, x.z, x.w, y.x, y.y, y.z, y.w}};
            }
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) v[tt][hh][ln].r[e] = 0u;
          }
        }
      }
  };
  auto score_tile = [&](const u32x8 (&v)[T][2][NLINE], int ptile) {
    const long long r0 = (long long)ptile * ROWS_PER_CTA + warp * 16 * T;
#pragma unroll
    for (int tt = 0; tt < T; ++tt) {
      float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int ln = 0; ln < NLINE; ++ln) {
        const u32x8 &lo = v[tt][0][ln], &hi = v[tt][1][ln];
#pragma unroll
        for (int m = 0; m < 4; ++m)
          mma_bf16_16816(c, lo.r[2 * m], hi.r[2 * m], lo.r[2 * m + 1], hi.r[2 * m + 1], bq[ln][m][0], bq[ln][m][1]);
      }
      // lane t4 = 0 holds the hi and mid column sums, t4 = 1 the lo sum (its second column is zero)
      float s0 = c[0] + c[1], s1 = c[2] + c[3];
      s0 += __shfl_xor_sync(0xffffffffu, s0, 1);
      s1 += __shfl_xor_sync(0xffffffffu, s1, 1);
      if (t4 == 0 && ptile < n_tiles) {
        const long long row = r0 + tt * 16 + grp;
        if (row < L) {
          wg[row] = s0;
          atomicAdd(&sh[order_key_f(s0) >> 20], 1);
        }
        if (row + 8 < L) {
          wg[row + 8] = s1;
          atomicAdd(&sh[order_key_f(s1) >> 20], 1);
        }
      }
    }
  };
  u32x8 va[T][2][NLINE], vb[T][2][NLINE];
  const int gx = (int)gridDim.x;
  load_tile(va, (int)blockIdx.x);
  for (int pt = (int)blockIdx.x; pt < n_tiles; pt += 2 * gx) {  // the bound does not depend on the lane: the shuffles see full warps
    load_tile(vb, pt + gx);
    score_tile(va, pt);
    load_tile(va, pt + 2 * gx);
    score_tile(vb, pt + gx);
  }
  __syncthreads();
  for (int b = threadIdx.x; b < HIST12; b += CMP_THREADS)
    if (sh[b]) atomicAdd(&hist12[g * HIST12 + b], sh[b]);
}

// exclusive scan of one int per thread over the CTA
__device__ int block_excl_scan_i(int v, int* warp_sums, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    const int ws = warp_sums[lane];
    int winc = ws;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    warp_sums[lane] = winc - ws;
    if (lane == 31) warp_sums[32] = winc;
  }
  __syncthreads();
  *total = warp_sums[32];
  return warp_sums[warp] + inc - v;
}

// one CTA per KV head: positions of the `keep` largest w, ascending; ties to the lower position.
// The top 12 key bits of the threshold come from the histogram the scoring pass left behind; the remaining
// 20 bits take three passes over w in which only the (few) keys sharing the known prefix touch the counters.
__global__ void __launch_bounds__(TOPK_THREADS, 1) topk_kernel(const float* w, const int* hist12,
                                                               int* __restrict__ idx, int L, int keep) {
  __shared__ int hist[256];
  __shared__ int s_scan[33];
  __shared__ uint32_t s_prefix;
  __shared__ int s_remaining;
  const int g = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* wg = w + (long long)g * L;
  int* out = idx + (long long)g * keep;
  chain_release();
  chain_wait();
  if (keep >= L) {
    for (int j = tid; j < L; j += TOPK_THREADS) out[j] = j;
    return;
  }
  // ---- 12 leading bits: thread t owns bins 4095-4t .. 4092-4t (descending); find the bin holding rank `keep`
  {
    const int* hg = hist12 + g * HIST12;
    int cnt[4], lsum = 0;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      cnt[t] = hg[HIST12 - 1 - 4 * tid - t];
      lsum += cnt[t];
    }
    int tot;
    const int excl = block_excl_scan_i(lsum, s_scan, &tot);
    if (excl < keep && excl + lsum >= keep) {
      int run = excl, bin = 0, above = 0;
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        if (run < keep && run + cnt[t] >= keep) {
          bin = HIST12 - 1 - 4 * tid - t;
          above = run;
        }
        run += cnt[t];
      }
      s_prefix = (uint32_t)bin << 20;
      s_remaining = keep - above;
    }
    __syncthreads();
  }
  uint32_t prefix = s_prefix, mask = 0xFFF00000u;
  int remaining = s_remaining;  // rank of the threshold among the keys matching the prefix (1-based from the top)
  __syncthreads();
  const int shifts[3] = {12, 4, 0}, widths[3] = {8, 8, 4};
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = shifts[pass], nb = 1 << widths[pass];
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    {
      auto count = [&](float f) {
        const uint32_t key = order_key_f(f);
        if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & (nb - 1)], 1);
      };
      const int L4 = L & ~3;
      const float4* w4 = reinterpret_cast<const float4*>(wg);  // wg is 16-byte aligned when L % 4 == 0 or g == 0
      const bool vec = ((reinterpret_cast<uintptr_t>(wg) & 15u) == 0);
      if (vec) {
        for (int b0 = tid; b0 < L4 / 4; b0 += TOPK_THREADS * 4) {  // four 16-byte loads in flight per thread
          float4 v[4];
#pragma unroll
          for (int u = 0; u < 4; ++u)
            if (b0 + u * TOPK_THREADS < L4 / 4) v[u] = w4[b0 + u * TOPK_THREADS];
#pragma unroll
          for (int u = 0; u < 4; ++u)
            if (b0 + u * TOPK_THREADS < L4 / 4) {
              count(v[u].x);
              count(v[u].y);
              count(v[u].z);
              count(v[u].w);
            }
        }
        for (int j = L4 + tid; j < L; j += TOPK_THREADS) count(wg[j]);
      } else {
        for (int j = tid; j < L; j += TOPK_THREADS) count(wg[j]);
      }
    }
    __syncthreads();
    if (warp == 0) {  // lane l owns bins nb-1-8l .. nb-8-8l (descending); bins beyond nb are empty
      int cnt[8], lsum = 0;
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const int b = nb - 1 - 8 * lane - t;
        cnt[t] = b >= 0 ? hist[b] : 0;
        lsum += cnt[t];
      }
      int inc = lsum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      const int excl = inc - lsum;
      if (excl < remaining && inc >= remaining) {
        int run = excl, digit = 0, above = 0;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          if (run < remaining && run + cnt[t] >= remaining) {
            digit = nb - 1 - 8 * lane - t;
            above = run;
          }
          run += cnt[t];
        }
        s_prefix = prefix | ((uint32_t)digit << shift);
        s_remaining = remaining - above;
      }
    }
    __syncthreads();
    prefix = s_prefix;
    remaining = s_remaining;
    mask |= (uint32_t)(nb - 1) << shift;
    __syncthreads();
  }
  // prefix is the threshold key: keep every key above it and the first `remaining` equal to it, in position
  // order.  Warp w owns the contiguous positions [w*seg, (w+1)*seg): coalesced reads, ballots give the order
  // inside a warp, two small scans over the 32 warps give each warp its output slot and its share of the ties.
  const uint32_t thr = prefix;
  const int seg = ((L + 31) / 32 + 31) & ~31;  // positions per warp, a multiple of 32
  const int p0 = warp * seg, p1 = min(L, p0 + seg);
  int n_eq = 0, n_gt = 0;
  for (int j0 = p0; j0 < p1; j0 += 128) {  // four loads in flight
    uint32_t key[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = j0 + u * 32 + lane;
      key[u] = j < p1 ? order_key_f(wg[j]) : 0u;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const bool valid = j0 + u * 32 + lane < p1;
      n_eq += __popc(__ballot_sync(0xffffffffu, valid && key[u] == thr));
      n_gt += __popc(__ballot_sync(0xffffffffu, valid && key[u] > thr));
    }
  }
  __shared__ int s_eq[32], s_gt[32], s_eqb[32], s_pos[32];
  if (lane == 0) {
    s_eq[warp] = n_eq;
    s_gt[warp] = n_gt;
  }
  __syncthreads();
  if (tid == 0) {
    int eqb = 0, pos = 0;
    for (int x = 0; x < 32; ++x) {
      s_eqb[x] = eqb;
      s_pos[x] = pos;
      int take = remaining - eqb;
      take = take < 0 ? 0 : (take > s_eq[x] ? s_eq[x] : take);
      pos += s_gt[x] + take;
      eqb += s_eq[x];
    }
  }
  __syncthreads();
  int pos = s_pos[warp], eq_seen = s_eqb[warp];
  for (int j0 = p0; j0 < p1; j0 += 32) {
    const int j = j0 + lane;
    const bool valid = j < p1;
    const uint32_t key = valid ? order_key_f(wg[j]) : 0u;
    const bool eq = valid && key == thr;
    const unsigned eqm = __ballot_sync(0xffffffffu, eq);
    const int eq_rank = eq_seen + __popc(eqm & ((1u << lane) - 1));
    const bool take = valid && (key > thr || (eq && eq_rank < remaining));
    const unsigned tm = __ballot_sync(0xffffffffu, take);
    if (take) out[pos + __popc(tm & ((1u << lane) - 1))] = j;
    pos += __popc(tm);
    eq_seen += __popc(eqm);
  }
}

// The same selection for L <= TKC_MAX_L, spread over a thread-block cluster per KV head: every thread keeps its
// TKC_VPT order keys in registers, so the scores are read once; the three radix histograms and the per-warp
// counts live in the shared memory of the cluster's first CTA and are reached through distributed shared memory.
// Warp x of CTA c owns the contiguous positions [c*chunk + x*seg, +seg), which keeps the output in position order.
constexpr int TKC_VPT = 16;
constexpr int TKC_MAX_CL = 8;
constexpr int TKC_MAX_L = TKC_MAX_CL * TOPK_THREADS * TKC_VPT;
__global__ void __launch_bounds__(TOPK_THREADS, 1) topk_cluster_kernel(const float* w, const int* hist12,
                                                                       int* __restrict__ idx_out, int L, int keep) {
  namespace cg = cooperative_groups;
  cg::cluster_group cl = cg::this_cluster();
  const int c = (int)cl.block_rank(), CL = (int)cl.num_blocks();
  __shared__ int hist[3][256];
  __shared__ int s_gt[TKC_MAX_CL * 32], s_eq[TKC_MAX_CL * 32];
  __shared__ int s_scan[32];
  __shared__ uint32_t s_prefix;
  __shared__ int s_remaining;
  const int g = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* wg = w + (size_t)g * L;
  int* out = idx_out + (size_t)g * keep;
  const int chunk = ((L + CL - 1) / CL + TOPK_THREADS - 1) & ~(TOPK_THREADS - 1);
  const int seg = chunk / 32;  // a multiple of 32, at most 32 * TKC_VPT
  const int p0 = c * chunk + warp * seg;
  chain_release();
  if (keep >= L) {  // the same branch in every CTA of the cluster
    for (int u = 0; u * 32 < seg; ++u) {
      const int j = p0 + u * 32 + lane;
      if (j < L) out[j] = j;
    }
    chain_wait();  // every link of the chain waits for the one before it, so that whatever follows this grid is
                   // also ordered after the scoring kernel's writes (w and its histogram)
    return;
  }
  for (int x = tid; x < 3 * 256; x += TOPK_THREADS) (&hist[0][0])[x] = 0;
  chain_wait();  // the scores and their histogram come from the kernel before
  uint32_t key[TKC_VPT];
  unsigned validm = 0;
#pragma unroll
  for (int u = 0; u < TKC_VPT; ++u) {
    const int j = p0 + u * 32 + lane;
    const bool ok = u * 32 < seg && j < L;
    key[u] = ok ? order_key_f(wg[j]) : 0u;
    validm |= (unsigned)ok << u;
  }
  {  // 12 leading bits from the histogram the scoring pass built; every CTA repeats this small step
    const int* hg = hist12 + g * HIST12;
    int cnt[4], lsum = 0;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      cnt[t] = hg[HIST12 - 1 - 4 * tid - t];
      lsum += cnt[t];
    }
    int tot;
    const int excl = block_excl_scan_i(lsum, s_scan, &tot);
    if (excl < keep && excl + lsum >= keep) {
      int run = excl, bin = 0, above = 0;
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        if (run < keep && run + cnt[t] >= keep) {
          bin = HIST12 - 1 - 4 * tid - t;
          above = run;
        }
        run += cnt[t];
      }
      s_prefix = (uint32_t)bin << 20;
      s_remaining = keep - above;
    }
  }
  cl.sync();  // histograms zeroed in the first CTA, s_prefix visible in this one
  uint32_t prefix = s_prefix, mask = 0xFFF00000u;
  int remaining = s_remaining;
  const int shifts[3] = {12, 4, 0}, widths[3] = {8, 8, 4};
#pragma unroll
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = shifts[pass], nb = 1 << widths[pass];
    int* rh = cl.map_shared_rank(&hist[pass][0], 0);
#pragma unroll
    for (int u = 0; u < TKC_VPT; ++u)
      if (((validm >> u) & 1u) && (key[u] & mask) == prefix) atomicAdd(&rh[(key[u] >> shift) & (nb - 1)], 1);
    cl.sync();
    if (warp == 0) {  // lane l owns bins nb-1-8l .. nb-8-8l (descending); bins beyond nb are empty
      int cnt[8], lsum = 0;
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const int b = nb - 1 - 8 * lane - t;
        cnt[t] = b >= 0 ? rh[b] : 0;
        lsum += cnt[t];
      }
      int inc = lsum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      const int excl = inc - lsum;
      if (excl < remaining && inc >= remaining) {
        int run = excl, digit = 0, above = 0;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          if (run < remaining && run + cnt[t] >= remaining) {
            digit = nb - 1 - 8 * lane - t;
            above = run;
          }
          run += cnt[t];
        }
        s_prefix = prefix | ((uint32_t)digit << shift);
        s_remaining = remaining - above;
      }
    }
    __syncthreads();
    prefix = s_prefix;
    remaining = s_remaining;
    mask |= (uint32_t)(nb - 1) << shift;
    __syncthreads();
  }
  // prefix is the threshold key: keep every key above it and the first `remaining` equal to it, in position order
  const uint32_t thr = prefix;
  int n_eq = 0, n_gt = 0;
#pragma unroll
  for (int u = 0; u < TKC_VPT; ++u) {
    const bool ok = (validm >> u) & 1u;
    n_eq += __popc(__ballot_sync(0xffffffffu, ok && key[u] == thr));
    n_gt += __popc(__ballot_sync(0xffffffffu, ok && key[u] > thr));
  }
  const int me = c * 32 + warp;  // this warp's place in position order over the cluster
  // every CTA gets its own copy of all warps' counts (lane x stores into CTA x), then scans it locally: reading
  // them all out of one CTA's shared memory made that CTA's port the bottleneck
  if (lane < CL) {
    cl.map_shared_rank(&s_gt[0], lane)[me] = n_gt;
    cl.map_shared_rank(&s_eq[0], lane)[me] = n_eq;
  }
  cl.sync();
  if (warp == 0) {
    int carry_eq = 0, carry_pos = 0;
    for (int x0 = 0; x0 < CL * 32; x0 += 32) {
      const int x = x0 + lane;
      const int e = s_eq[x], gt = s_gt[x];
      int inc = e;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      const int eqb = carry_eq + inc - e;  // ties in the warps before x
      int take = remaining - eqb;
      take = take < 0 ? 0 : (take > e ? e : take);
      int pinc = gt + take;
      const int mine = pinc;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, pinc, o);
        if (lane >= o) pinc += t;
      }
      s_eq[x] = eqb;                       // from here on: ties before warp x
      s_gt[x] = carry_pos + pinc - mine;   // from here on: output slot of warp x
      carry_eq += __shfl_sync(0xffffffffu, inc, 31);
      carry_pos += __shfl_sync(0xffffffffu, pinc, 31);
    }
  }
  __syncthreads();
  int pos = s_gt[me], eq_seen = s_eq[me];
#pragma unroll
  for (int u = 0; u < TKC_VPT; ++u) {
    const bool ok = (validm >> u) & 1u;
    const bool eq = ok && key[u] == thr;
    const unsigned eqm = __ballot_sync(0xffffffffu, eq);
    const int eq_rank = eq_seen + __popc(eqm & ((1u << lane) - 1));
    const bool take = ok && (key[u] > thr || (eq && eq_rank < remaining));
    const unsigned tm = __ballot_sync(0xffffffffu, take);
    if (take) out[pos + __popc(tm & ((1u << lane) - 1))] = p0 + u * 32 + lane;
    pos += __popc(tm);
    eq_seen += __popc(eqm);
  }
  // the last access to another CTA's shared memory is before the cluster barrier above, so CTAs may leave freely
}

// K_out[g, t, :] = K[g, idx[g,t], :] (and V): LPR 16-byte lanes per row
template <int D>
__global__ void __launch_bounds__(CMP_THREADS) gather_kernel(const __nv_bfloat16* __restrict__ k,
                                                             const __nv_bfloat16* __restrict__ v,
                                                             const int* idx, __nv_bfloat16* __restrict__ ko,
                                                             __nv_bfloat16* __restrict__ vo, int keep, long long ks_h,
                                                             long long ks_t, long long vs_h, long long vs_t) {
  constexpr int LPR = D / 8;
  const int g = blockIdx.y;
  const int lane16 = threadIdx.x % LPR;
  const int t = blockIdx.x * (CMP_THREADS / LPR) + threadIdx.x / LPR;
  chain_wait();  // idx comes from the kernel before
  if (t >= keep) return;
  const int j = idx[(long long)g * keep + t];
  const uint4 a = *reinterpret_cast<const uint4*>(k + (long long)g * ks_h + (long long)j * ks_t + lane16 * 8);
  const uint4 b = *reinterpret_cast<const uint4*>(v + (long long)g * vs_h + (long long)j * vs_t + lane16 * 8);
  reinterpret_cast<uint4*>(ko + ((long long)g * keep + t) * D)[lane16] = a;
  reinterpret_cast<uint4*>(vo + ((long long)g * keep + t) * D)[lane16] = b;
}

}  // namespace

}  // namespace ei

namespace ei {
namespace {
// launch as a link of the chain: may start before the kernel ahead of it in the stream has finished
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kern)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, unsigned cluster_x,
                           bool early, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = early ? 1 : 0;
  cfg.numAttrs = 1;
  if (cluster_x) {
    at[1].id = cudaLaunchAttributeClusterDimension;
    at[1].val.clusterDim.x = cluster_x;
    at[1].val.clusterDim.y = 1;
    at[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  cfg.attrs = at;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
}  // namespace
}  // namespace ei

extern "C" {

size_t ei_latent_compress_workspace_bytes(const ei_compress_params* p) {
  if (!p || p->struct_size != sizeof(ei_compress_params) || p->n_kv_heads <= 0 || p->kv_len <= 0 || p->head_dim <= 0)
    return 0;
  return sizeof(float) * ((size_t)p->n_kv_heads * (size_t)p->kv_len + (size_t)p->n_kv_heads * (size_t)p->head_dim) +
         sizeof(int) * (size_t)p->n_kv_heads * ei::HIST12;
}

int ei_latent_compress(const ei_compress_params* p, const void* q_window, const void* k, const void* v,
                       void* workspace, int32_t* idx_out, void* k_out, void* v_out, void* stream) {
  if (!p || p->struct_size != sizeof(ei_compress_params)) return EI_ERR_INVALID_ARG;
  if (!q_window || !k || !v || !workspace || !idx_out || !k_out || !v_out) return EI_ERR_INVALID_ARG;
  if (p->n_q_heads <= 0 || p->n_kv_heads <= 0 || p->kv_len <= 0 || p->window <= 0 || p->budget <= 0)
    return EI_ERR_INVALID_ARG;
  if ((p->head_dim != 64 && p->head_dim != 128 && p->head_dim != 256) || p->n_q_heads % p->n_kv_heads)
    return EI_ERR_UNSUPPORTED_SHAPE;
  const int64_t strides[6] = {p->q_stride_head, p->q_stride_tok, p->k_stride_head,
                              p->k_stride_tok,  p->v_stride_head, p->v_stride_tok};
  for (int64_t s : strides)
    if (s < p->head_dim || s % 8) return EI_ERR_UNSUPPORTED_SHAPE;
  const uintptr_t al = reinterpret_cast<uintptr_t>(q_window) | reinterpret_cast<uintptr_t>(k) |
                       reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(workspace) |
                       reinterpret_cast<uintptr_t>(k_out) | reinterpret_cast<uintptr_t>(v_out);
  if (al & 15u) return EI_ERR_UNSUPPORTED_SHAPE;

  const int Hkv = p->n_kv_heads, G = p->n_q_heads / Hkv, d = p->head_dim, L = p->kv_len;
  const int keep = p->budget < L ? p->budget : L;
  cudaStream_t st = (cudaStream_t)stream;
  float* w = static_cast<float*>(workspace);
  float* qsum = w + (size_t)Hkv * L;
  int* hist12 = reinterpret_cast<int*>(qsum + (size_t)Hkv * d);
  const __nv_bfloat16* kk = static_cast<const __nv_bfloat16*>(k);
  const __nv_bfloat16* vv = static_cast<const __nv_bfloat16*>(v);
  const __nv_bfloat16* qq = static_cast<const __nv_bfloat16*>(q_window);
  __nv_bfloat16* ko = static_cast<__nv_bfloat16*>(k_out);
  __nv_bfloat16* vo = static_cast<__nv_bfloat16*>(v_out);

  // head of the chain: an ordinary launch, ordered after everything already in the stream
  if (d == 256)
    ei::qsum_kernel<256><<<Hkv, ei::CMP_THREADS, 0, st>>>(qq, qsum, hist12, G, p->window, p->q_stride_head, p->q_stride_tok);
  else if (d == 128)
    ei::qsum_kernel<128><<<Hkv, ei::CMP_THREADS, 0, st>>>(qq, qsum, hist12, G, p->window, p->q_stride_head, p->q_stride_tok);
  else
    ei::qsum_kernel<64><<<Hkv, ei::CMP_THREADS, 0, st>>>(qq, qsum, hist12, G, p->window, p->q_stride_head, p->q_stride_tok);
  const int tiles_in_flight = SCORE_TILES * 128 / d > 0 ? SCORE_TILES * 128 / d : 1;
  const int rows_per_cta = (ei::CMP_THREADS / 32) * 16 * tiles_in_flight;
  // four resident CTAs per SM in all, the CTAs of grid row y on head y: the fastest of the shapes measured (one
  // sequence over all heads, where every CTA hands over a histogram per head, was about twice slower)
  int gx = (L + rows_per_cta - 1) / rows_per_cta;
  const int gx_cap = (148 * SCORE_CTAS_PER_SM + Hkv - 1) / Hkv;
  if (gx > gx_cap) gx = gx_cap;
  const dim3 sgrid((unsigned)gx, (unsigned)Hkv), blk(ei::CMP_THREADS);
  const dim3 ggrid((unsigned)((keep + ei::CMP_THREADS / (d / 8) - 1) / (ei::CMP_THREADS / (d / 8))), (unsigned)Hkv);
  const bool wide = ((reinterpret_cast<uintptr_t>(k) | (uintptr_t)(p->k_stride_head * 2) | (uintptr_t)(p->k_stride_tok * 2)) & 31u) == 0;
  auto score = d == 256   ? (wide ? ei::score_kernel<256, true> : ei::score_kernel<256, false>)
               : d == 128 ? (wide ? ei::score_kernel<128, true> : ei::score_kernel<128, false>)
                          : (wide ? ei::score_kernel<64, true> : ei::score_kernel<64, false>);
  if (ei::launch_chained(score, sgrid, blk, st, 0u, true, kk, qsum, w, hist12, L, Hkv, (long long)p->k_stride_head,
                         (long long)p->k_stride_tok) != cudaSuccess)
    return EI_ERR_CUDA;
  cudaError_t e;
  if (L <= ei::TKC_MAX_L) {
    const int per_cta = ei::TOPK_THREADS * ei::TKC_VPT;
    const unsigned CL = (unsigned)((L + per_cta - 1) / per_cta);
    e = ei::launch_chained(ei::topk_cluster_kernel, dim3(CL, (unsigned)Hkv), dim3(ei::TOPK_THREADS), st, CL, true, w, hist12,
                           idx_out, L, keep);
  } else {
    e = ei::launch_chained(ei::topk_kernel, dim3((unsigned)Hkv), dim3(ei::TOPK_THREADS), st, 0u, true, w, hist12, idx_out, L,
                           keep);
  }
  if (e != cudaSuccess) return EI_ERR_CUDA;
  auto gather = d == 256 ? ei::gather_kernel<256> : d == 128 ? ei::gather_kernel<128> : ei::gather_kernel<64>;
  if (ei::launch_chained(gather, ggrid, blk, st, 0u, true, kk, vv, idx_out, ko, vo, keep, (long long)p->k_stride_head,
                         (long long)p->k_stride_tok, (long long)p->v_stride_head, (long long)p->v_stride_tok) !=
      cudaSuccess)
    return EI_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

}  // extern "C"
