// Planning kernels of the EntropyInfer prefill path (stages 1-3), sm_100a.
//
//   pool_kernel     Alg. 1   elementwise max/min of Q per segment and of K per key block (HBM-bound)
//   observe_kernel  Alg. 2   four pooled logit matrices, causal row softmax, A_obs, ln A_obs,
//                            and the row entropy e[h,i] = -sum_j A ln A
//   budget_kernel   Alg. 3   head class, budget multipliers, block counts (exact integer
//                            apportionment to a configured total), CSR offsets
//   select_kernel   Eq. t_topk   per (head, segment) top-(k - r) blocks by ln A_obs, ties to the
//                            lower index, diagonal blocks appended, ascending output
#include <math.h>

#include "ei_internal.cuh"
#include "ei_sm100.cuh"

namespace ei {

// =================================================================================================
// Stage 1a -- pooling (Alg. 1).  One CTA per cell: a (query head, segment) of L_S rows or a
// (KV head, key block) of L_B rows.  Each row is D bf16 = D/8 16-byte lanes; 256 threads cover
// 256/(D/8) rows per pass with coalesced, streaming 16-byte loads.  max/min of bf16 are exact.
// =================================================================================================
__device__ __forceinline__ uint4 ld_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ uint32_t bmax2(uint32_t a, uint32_t b) {
  __nv_bfloat162 r = __hmax2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
  return *reinterpret_cast<uint32_t*>(&r);
}
__device__ __forceinline__ uint32_t bmin2(uint32_t a, uint32_t b) {
  __nv_bfloat162 r = __hmin2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
  return *reinterpret_cast<uint32_t*>(&r);
}
__device__ __forceinline__ void acc_max(uint4& m, const uint4& v) {
  m.x = bmax2(m.x, v.x); m.y = bmax2(m.y, v.y); m.z = bmax2(m.z, v.z); m.w = bmax2(m.w, v.w);
}
__device__ __forceinline__ void acc_min(uint4& m, const uint4& v) {
  m.x = bmin2(m.x, v.x); m.y = bmin2(m.y, v.y); m.z = bmin2(m.z, v.z); m.w = bmin2(m.w, v.w);
}

template <int D>
__global__ void __launch_bounds__(256) pool_kernel(const __nv_bfloat16* __restrict__ q,
                                                   const __nv_bfloat16* __restrict__ k,
                                                   __nv_bfloat16* __restrict__ qmax,
                                                   __nv_bfloat16* __restrict__ qmin,
                                                   __nv_bfloat16* __restrict__ kmax,
                                                   __nv_bfloat16* __restrict__ kmin, Shape s, long long cell0,
                                                   int kb0, const PackedSeq* pk, int npk) {
  constexpr int LPR = D / 8;     // 16-byte lanes per row
  constexpr int RS = 256 / LPR;  // rows per pass
  constexpr int UNROLL = 8;
  __shared__ uint4 smx[256];
  __shared__ uint4 smn[256];

  const int tid = threadIdx.x;
  const int lane16 = tid % LPR, slot = tid / LPR;
  int bid = blockIdx.x;
  if (pk != nullptr) {  // a packed batch: my sequence's shape, my CTA's number within it, its share of the tables
    const PackedSeq& P = pk[packed_find(pk, npk, bid, &PackedSeq::w_pool)];
    s = P.s;
    bid -= P.w_pool;
    q += P.tok0 * s.qs_t;
    k += P.tok0 * s.ks_t;
    qmax += P.cell0 * D;
    qmin += P.cell0 * D;
    kmax += P.kb0 * D;
    kmin += P.kb0 * D;
  }
  long long cell = cell0 + bid;  // cell0 = s.cells pools the K blocks only
  const __nv_bfloat16* base;
  long long tok_stride;
  int L;
  __nv_bfloat16 *omax, *omin;
  if (cell < s.cells) {
    const long long h = cell / s.C_S, i = cell % s.C_S;
    base = q + h * s.qs_h + i * s.L_S * s.qs_t;
    tok_stride = s.qs_t;
    L = (int)min((long long)s.L_S, s.Nq - i * s.L_S);  // a short last segment is pooled over the rows it has
    omax = qmax + cell * D;
    omin = qmin + cell * D;
  } else {
    cell -= s.cells;
    const long long nb = s.C_B - kb0;  // key blocks pooled per KV head: [kb0, C_B)
    const long long g = cell / nb, j = kb0 + cell % nb;
    base = k + g * s.ks_h + j * s.L_B * s.ks_t;
    tok_stride = s.ks_t;
    L = (int)min((long long)s.L_B, s.N - j * s.L_B);
    omax = kmax + (g * s.KB_cap + j) * D;
    omin = kmin + (g * s.KB_cap + j) * D;
  }
  const uint32_t NEG = 0xFF80FF80u, POS = 0x7F807F80u;  // bf16x2 -inf / +inf
  uint4 mx = make_uint4(NEG, NEG, NEG, NEG), mn = make_uint4(POS, POS, POS, POS);
  const __nv_bfloat16* p = base + lane16 * 8;
  for (int row0 = slot; row0 < L; row0 += RS * UNROLL) {
    uint4 v[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int row = row0 + u * RS;
      if (row < L) v[u] = ld_stream(p + (long long)row * tok_stride);
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int row = row0 + u * RS;
      if (row < L) {
        acc_max(mx, v[u]);
        acc_min(mn, v[u]);
      }
    }
  }
  smx[tid] = mx;
  smn[tid] = mn;
  __syncthreads();
#pragma unroll
  for (int half = RS / 2; half > 0; half >>= 1) {
    if (slot < half) {
      uint4 a = smx[tid], b = smx[tid + half * LPR];
      acc_max(a, b);
      smx[tid] = a;
      a = smn[tid];
      b = smn[tid + half * LPR];
      acc_min(a, b);
      smn[tid] = a;
    }
    __syncthreads();
  }
  if (slot == 0) {
    reinterpret_cast<uint4*>(omax)[lane16] = smx[tid];
    reinterpret_cast<uint4*>(omin)[lane16] = smn[tid];
  }
}

cudaError_t launch_pool(const Shape& s, const __nv_bfloat16* q, const __nv_bfloat16* k,
                        __nv_bfloat16* qmax, __nv_bfloat16* qmin, __nv_bfloat16* kmax,
                        __nv_bfloat16* kmin, int first_block, cudaStream_t st) {
  const long long grid = s.cells + (long long)s.Hkv * max(0, s.C_B - first_block);
  if (s.d == 256)
    pool_kernel<256><<<(unsigned)grid, 256, 0, st>>>(q, k, qmax, qmin, kmax, kmin, s, 0, first_block, nullptr, 0);
  else if (s.d == 128)
    pool_kernel<128><<<(unsigned)grid, 256, 0, st>>>(q, k, qmax, qmin, kmax, kmin, s, 0, first_block, nullptr, 0);
  else
    pool_kernel<64><<<(unsigned)grid, 256, 0, st>>>(q, k, qmax, qmin, kmax, kmin, s, 0, first_block, nullptr, 0);
  return cudaGetLastError();
}

cudaError_t launch_pool_packed(const PackedSeq* pk, const PackedSeq* pk_host, int npk, const __nv_bfloat16* q,
                               const __nv_bfloat16* k, __nv_bfloat16* qmax, __nv_bfloat16* qmin, __nv_bfloat16* kmax,
                               __nv_bfloat16* kmin, cudaStream_t st) {
  const Shape& s = pk_host[npk - 1].s;
  const long long grid = pk_host[npk - 1].w_pool + s.cells + (long long)s.Hkv * s.C_B;
  if (s.d == 256)
    pool_kernel<256><<<(unsigned)grid, 256, 0, st>>>(q, k, qmax, qmin, kmax, kmin, s, 0, 0, pk, npk);
  else if (s.d == 128)
    pool_kernel<128><<<(unsigned)grid, 256, 0, st>>>(q, k, qmax, qmin, kmax, kmin, s, 0, 0, pk, npk);
  else
    pool_kernel<64><<<(unsigned)grid, 256, 0, st>>>(q, k, qmax, qmin, kmax, kmin, s, 0, 0, pk, npk);
  return cudaGetLastError();
}

cudaError_t launch_pool_k(const Shape& s, const __nv_bfloat16* k, __nv_bfloat16* kmax, __nv_bfloat16* kmin,
                          int first_block, cudaStream_t st) {
  const long long grid = (long long)s.Hkv * (s.C_B - first_block);
  if (grid <= 0) return cudaSuccess;
  if (s.d == 256)
    pool_kernel<256><<<(unsigned)grid, 256, 0, st>>>(nullptr, k, nullptr, nullptr, kmax, kmin, s, s.cells, first_block, nullptr, 0);
  else if (s.d == 128)
    pool_kernel<128><<<(unsigned)grid, 256, 0, st>>>(nullptr, k, nullptr, nullptr, kmax, kmin, s, s.cells, first_block, nullptr, 0);
  else
    pool_kernel<64><<<(unsigned)grid, 256, 0, st>>>(nullptr, k, nullptr, nullptr, kmax, kmin, s, s.cells, first_block, nullptr, 0);
  return cudaGetLastError();
}

// =================================================================================================
// Stage 1b -- observation attention and entropy (Alg. 2, entropy definition).
// One CTA per (KV head g, segment i, sub-group of up to HG query heads of the group): the K
// representatives of the row's C_i = r(i+1) causal blocks are read once and used for all HG
// heads (one warp per key block, lanes split the head dimension, butterfly reduction).
// Dot products are accumulated in fp64 (products of bf16 are exact), the four logits of
// every (head, block) stay in shared memory as fp64, and only exp/log of bounded arguments run
// in fp32.  ln A is formed in the log domain:
//     l_m = x_m - logsumexp_j(x_m),  lnA = max(logaddexp(l1,l2), logaddexp(l3,l4)) - ln 2
// so that entries far below fp32 range still rank by value; lnA is clamped to <= 0 (each
// softmax value is <= 1).  e = -sum_j exp(lnA) * lnA, not renormalised.
// =================================================================================================
constexpr int OBS_THREADS = 512;
constexpr int OBS_WARPS = OBS_THREADS / 32;

__device__ __forceinline__ double warp_max_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// bf16 -> fp64 with integer instructions only (keeps the conversions off the special-function / MIO path
// that the shared-memory broadcasts also use).  h is the bf16 pattern in the low 16 bits.  Exact for
// normal numbers and zero; bf16 subnormals (|x| < 1.2e-38) are flushed to zero, which cannot change a
// logit by more than 1e-36.
__device__ __forceinline__ double bf16_to_f64(uint32_t h) {
  const uint32_t sign = (h & 0x8000u) << 16;
  const uint32_t em = h & 0x7FFFu;                              // exponent (8) | mantissa (7)
  const uint32_t hi = (em >= 0x80u) ? (sign | ((em << 13) + (896u << 20))) : sign;  // rebias 127 -> 1023
  return __hiloint2double((int)hi, 0);
}
__device__ __forceinline__ double bf16lo(uint32_t w) { return bf16_to_f64(w & 0xFFFFu); }
__device__ __forceinline__ double bf16hi(uint32_t w) { return bf16_to_f64(w >> 16); }
// the same conversions through the fp32 -> fp64 convert instruction (exact as well); the observation kernel
// uses both kinds so that neither the integer pipe nor the conversion pipe becomes the limiter
__device__ __forceinline__ double bf16lo_cvt(uint32_t w) { return (double)__uint_as_float(w << 16); }
__device__ __forceinline__ double bf16hi_cvt(uint32_t w) { return (double)__uint_as_float(w & 0xFFFF0000u); }

template <int D, int HG>
__global__ void __launch_bounds__(OBS_THREADS, 1)
observe_kernel(const __nv_bfloat16* __restrict__ qmax, const __nv_bfloat16* __restrict__ qmin,
               const __nv_bfloat16* __restrict__ kmax, const __nv_bfloat16* __restrict__ kmin,
               float* __restrict__ scores, float* __restrict__ entropy, Shape s, double scale,
               int nsub, int xcap, const PackedSeq* pk, int npk) {
  extern __shared__ __align__(16) unsigned char obs_smem[];
  // layout: lse [HG*4] double | epart [HG][OBS_WARPS] double | xs [HG*4][xcap] double
  double* lse = reinterpret_cast<double*>(obs_smem);
  double* epart = lse + HG * 4;
  double* xs = epart + HG * OBS_WARPS;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // longest rows first
  int bid = blockIdx.x;
  if (pk != nullptr) {  // a packed batch: my sequence's shape, my CTA's number within it, its share of the tables
    const PackedSeq& P = pk[packed_find(pk, npk, bid, &PackedSeq::w_obs)];
    s = P.s;
    bid -= P.w_obs;
    qmax += P.cell0 * D;
    qmin += P.cell0 * D;
    kmax += P.kb0 * D;
    kmin += P.kb0 * D;
    scores += P.sc0;
    entropy += P.cell0;
  }
  const int sub = bid % nsub;
  bid /= nsub;
  const int g = bid % s.Hkv;
  const int i = s.C_S - 1 - bid / s.Hkv;
  const int Ci = causal_blocks(s, i);
  const int h0 = g * s.G + sub * HG;
  const int nh = min(HG, s.G - sub * HG);  // heads handled here (last sub-group may be short)

  // ---- phase 1: logits ---------------------------------------------------------------------
  // The logits of a row are a small matrix product: [HG*2 query representatives] x [2*C_i key
  // representatives] over d, in fp64.  It runs on the fp64 matrix instruction (m8n8k4): eight query
  // rows (up to four heads x max/min) x eight key vectors (four blocks x max/min) per warp-level step.
  // A lane keeps its share of the query matrix in registers for the whole CTA, reads 16 contiguous
  // bytes of a key representative per 8 instructions, and needs neither shared-memory broadcasts nor
  // shuffles.  The order in which d is walked is permuted the same way for both operands (lane c of a
  // quad takes elements 8*(c + 4s) .. +7 in super-step s), which leaves every dot product unchanged.
  // A head dimension above 128 is walked in passes of 128 elements (the query operand of one pass fills the
  // register budget); the partial sums of a pass wait in shared memory, written and re-read by the same thread.
  constexpr int DH = D > 128 ? 128 : D;
  constexpr int NPASS = D / DH;
  constexpr int NSS = DH / 32;  // super-steps of 32 elements
  const int qrow = lane >> 2, qc = lane & 3;  // A / C row (query vector), position in the quad
#pragma unroll 1
  for (int pass = 0; pass < NPASS; ++pass) {
    double qreg[NSS * 8];
    {
      const int hh = qrow >> 1, wq = qrow & 1;
      const bool valid = hh < nh && hh < HG;
      const __nv_bfloat16* src = (wq ? qmin : qmax) + ((long long)(h0 + (valid ? hh : 0)) * s.C_S + i) * D + pass * DH;
#pragma unroll
      for (int ss = 0; ss < NSS; ++ss) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(src + 8 * (qc + 4 * ss)));
        const double q8[8] = {bf16lo(v.x), bf16hi(v.x), bf16lo(v.y), bf16hi(v.y), bf16lo(v.z), bf16hi(v.z), bf16lo(v.w), bf16hi(v.w)};
#pragma unroll
        for (int t = 0; t < 8; ++t) qreg[ss * 8 + t] = valid ? q8[t] : 0.0;
      }
    }
    // two independent groups of four key blocks per warp step (two accumulator chains in flight)
    for (int j0 = warp * 8; j0 < Ci; j0 += OBS_WARPS * 8) {
      // B column n = lane / 4: key vector n -> block j0 (+4) + n/2 (clamped in the ragged tail), max or min
      const int jbA = min(j0 + (qrow >> 1), Ci - 1), jbB = min(j0 + 4 + (qrow >> 1), Ci - 1);
      const __nv_bfloat16* kbase = ((qrow & 1) ? kmin : kmax) + (long long)g * s.KB_cap * D + pass * DH;
      const __nv_bfloat16* krowA = kbase + (long long)jbA * D;
      const __nv_bfloat16* krowB = kbase + (long long)jbB * D;
      double a0 = 0.0, a1 = 0.0, b0 = 0.0, b1 = 0.0;
#pragma unroll
      for (int ss = 0; ss < NSS; ++ss) {
        const uint4 va = __ldg(reinterpret_cast<const uint4*>(krowA + 8 * (qc + 4 * ss)));
        const uint4 vb = __ldg(reinterpret_cast<const uint4*>(krowB + 8 * (qc + 4 * ss)));
        const double ka[8] = {bf16lo(va.x), bf16hi_cvt(va.x), bf16lo(va.y), bf16hi_cvt(va.y),
                              bf16lo(va.z), bf16hi_cvt(va.z), bf16lo(va.w), bf16hi_cvt(va.w)};
        const double kb[8] = {bf16lo(vb.x), bf16hi_cvt(vb.x), bf16lo(vb.y), bf16hi_cvt(vb.y),
                              bf16lo(vb.z), bf16hi_cvt(vb.z), bf16lo(vb.w), bf16hi_cvt(vb.w)};
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                       : "+d"(a0), "+d"(a1)
                       : "d"(qreg[ss * 8 + t]), "d"(ka[t]));
          asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                       : "+d"(b0), "+d"(b1)
                       : "d"(qreg[ss * 8 + t]), "d"(kb[t]));
        }
      }
      // C[row = query vector qrow][cols 2*qc, 2*qc+1] = key vectors of block j + qc: (Kmax, Kmin)
      const int hh = qrow >> 1, wq = qrow & 1;
      if (hh < HG) {
        const int jwA = j0 + qc, jwB = j0 + 4 + qc;
        double* x0 = xs + (size_t)(hh * 4 + wq * 2 + 0) * xcap;
        double* x1 = xs + (size_t)(hh * 4 + wq * 2 + 1) * xcap;
        if (NPASS > 1 && pass > 0) {
          if (jwA < Ci) { a0 += x0[jwA]; a1 += x1[jwA]; }
          if (jwB < Ci) { b0 += x0[jwB]; b1 += x1[jwB]; }
        }
        const double f = (pass == NPASS - 1) ? scale : 1.0;  // the last pass leaves the scaled logit
        if (jwA < Ci) {
          x0[jwA] = f * a0;
          x1[jwA] = f * a1;
        }
        if (jwB < Ci) {
          x0[jwB] = f * b0;
          x1[jwB] = f * b1;
        }
      }
    }
  }
  __syncthreads();

  // ---- phase 2: log-sum-exp of each (head, m) row -------------------------------------------
  for (int p = warp; p < nh * 4; p += OBS_WARPS) {
    const double* x = xs + p * xcap;
    double mx = -INFINITY;
    for (int j = lane; j < Ci; j += 32) mx = fmax(mx, x[j]);
    mx = warp_max_d(mx);
    float sum = 0.f;
    for (int j = lane; j < Ci; j += 32) sum += expf((float)(x[j] - mx));
    sum = warp_sum_f(sum);
    if (lane == 0) lse[p] = mx + (double)logf(sum);
  }
  __syncthreads();

  // ---- phase 3: ln A, scores out, entropy ---------------------------------------------------
  const double LN2 = 0.693147180559945309417232121458;
  for (int hh = 0; hh < nh; ++hh) {
    const double l0 = lse[hh * 4 + 0], l1 = lse[hh * 4 + 1], l2 = lse[hh * 4 + 2], l3 = lse[hh * 4 + 3];
    float* out = scores + (long long)(h0 + hh) * s.SC + row_offset(s, i);
    double e = 0.0;
    for (int j = tid; j < Ci; j += OBS_THREADS) {
      const double a1 = xs[(hh * 4 + 0) * xcap + j] - l0, a2 = xs[(hh * 4 + 1) * xcap + j] - l1;
      const double a3 = xs[(hh * 4 + 2) * xcap + j] - l2, a4 = xs[(hh * 4 + 3) * xcap + j] - l3;
      const double hi12 = fmax(a1, a2), lo12 = fmin(a1, a2);
      const double hi34 = fmax(a3, a4), lo34 = fmin(a3, a4);
      const double u = hi12 + (double)log1pf(expf((float)(lo12 - hi12)));
      const double w = hi34 + (double)log1pf(expf((float)(lo34 - hi34)));
      double l = fmin(fmax(u, w) - LN2, 0.0);
      const float lf = (float)l;
      out[j] = lf + 0.0f;  // canonical zero
      e -= (double)expf(lf) * l;
    }
    e = warp_sum_d(e);
    if (lane == 0) epart[hh * OBS_WARPS + warp] = e;
  }
  __syncthreads();
  if (tid < nh) {
    double e = 0.0;
    for (int w = 0; w < OBS_WARPS; ++w) e += epart[tid * OBS_WARPS + w];
    entropy[(long long)(h0 + tid) * s.C_S + i] = (float)e;
  }
}

static size_t observe_smem_bytes(int d, int hg, int xcap) {
  (void)d;
  return sizeof(double) * ((size_t)hg * 4 + (size_t)hg * OBS_WARPS + (size_t)hg * 4 * xcap);
}
static const size_t OBS_SMEM_LIMIT = 200 * 1024;

static int observe_pick_hg(const Shape& s) {
  for (int hg : {4, 2, 1}) {
    if (hg > s.G && hg != 1) continue;
    if (observe_smem_bytes(s.d, hg, s.C_B) <= OBS_SMEM_LIMIT) return hg;
  }
  return 0;
}
bool observe_shape_supported(const Shape& s) { return observe_pick_hg(s) != 0; }

template <int D, int HG>
static cudaError_t launch_observe_t(const Shape& s, const __nv_bfloat16* qmax, const __nv_bfloat16* qmin,
                                    const __nv_bfloat16* kmax, const __nv_bfloat16* kmin, double scale,
                                    float* scores, float* entropy, cudaStream_t st, const PackedSeq* pk = nullptr,
                                    int npk = 0, long long packed_grid = 0) {
  // (packed: s is the sequence with the most key blocks -- it sizes the shared-memory staging -- and the grid
  //  covers all sequences, w_obs counting C_S * H_kv * nsub CTAs per sequence)
  const int nsub = (s.G + HG - 1) / HG;
  const size_t smem = observe_smem_bytes(D, HG, s.C_B);
  cudaError_t e = cudaFuncSetAttribute(observe_kernel<D, HG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const unsigned grid = (unsigned)(pk ? packed_grid * nsub : (long long)s.C_S * s.Hkv * nsub);
  observe_kernel<D, HG><<<grid, OBS_THREADS, smem, st>>>(qmax, qmin, kmax, kmin, scores, entropy, s, scale, nsub, s.C_B,
                                                         pk, npk);
  return cudaGetLastError();
}

int observe_ctas_per_row(const Shape& s) {  // CTAs per (KV head, segment) row: the head sub-groups
  const int hg = observe_pick_hg(s);
  return hg ? (s.G + hg - 1) / hg : 0;
}

static cudaError_t launch_observe_any(const Shape& s, const __nv_bfloat16* qmax, const __nv_bfloat16* qmin,
                                      const __nv_bfloat16* kmax, const __nv_bfloat16* kmin, double scale, float* scores,
                                      float* entropy, cudaStream_t st, const PackedSeq* pk, int npk, long long packed_rows);

cudaError_t launch_observe(const Shape& s, const __nv_bfloat16* qmax, const __nv_bfloat16* qmin,
                           const __nv_bfloat16* kmax, const __nv_bfloat16* kmin, double scale,
                           float* scores, float* entropy, cudaStream_t st) {
  return launch_observe_any(s, qmax, qmin, kmax, kmin, scale, scores, entropy, st, nullptr, 0, 0);
}

// pk_host[i].w_obs counts (KV head, segment) ROWS of the earlier sequences times the CTAs per row
cudaError_t launch_observe_packed(const PackedSeq* pk, const PackedSeq* pk_host, int npk, const __nv_bfloat16* qmax,
                                  const __nv_bfloat16* qmin, const __nv_bfloat16* kmax, const __nv_bfloat16* kmin,
                                  double scale, float* scores, float* entropy, cudaStream_t st) {
  int big = 0;
  long long rows = 0;
  for (int i = 0; i < npk; ++i) {
    if (pk_host[i].s.C_B > pk_host[big].s.C_B) big = i;
    rows += (long long)pk_host[i].s.C_S * pk_host[i].s.Hkv;
  }
  return launch_observe_any(pk_host[big].s, qmax, qmin, kmax, kmin, scale, scores, entropy, st, pk, npk, rows);
}

static cudaError_t launch_observe_any(const Shape& s, const __nv_bfloat16* qmax, const __nv_bfloat16* qmin,
                                      const __nv_bfloat16* kmax, const __nv_bfloat16* kmin, double scale, float* scores,
                                      float* entropy, cudaStream_t st, const PackedSeq* pk, int npk, long long packed_rows) {
  const int hg = observe_pick_hg(s);
#define EI_OBS(D_, HG_) return launch_observe_t<D_, HG_>(s, qmax, qmin, kmax, kmin, scale, scores, entropy, st, pk, npk, packed_rows)
  if (s.d == 256) {
    if (hg == 4) EI_OBS(256, 4);
    if (hg == 2) EI_OBS(256, 2);
    if (hg == 1) EI_OBS(256, 1);
  } else if (s.d == 128) {
    if (hg == 4) EI_OBS(128, 4);
    if (hg == 2) EI_OBS(128, 2);
    if (hg == 1) EI_OBS(128, 1);
  } else {
    if (hg == 4) EI_OBS(64, 4);
    if (hg == 2) EI_OBS(64, 2);
    if (hg == 1) EI_OBS(64, 1);
  }
#undef EI_OBS
  return cudaErrorInvalidValue;
}

// =================================================================================================
// Stages 1a (queries) + 1b in one persistent kernel.  Pooling Q is bound by HBM, the observation by the
// fp64 matrix pipe, and neither leaves room for a second CTA on an SM, so run back to back they add up.
// Here a CTA of 32 warps walks a list of (KV head, segment, head sub-group) rows: warps 16-31 pool the
// query cells of the row after next into fp64 representatives in shared memory (and write the bf16
// representatives out as the pooling kernel does), while warps 0-15 run the observation of the current
// row exactly as observe_kernel does, reading the query operand of the matrix instruction from those
// shared-memory representatives instead of registers.  Two representative buffers, two mbarriers each way;
// every wait is bounded and reports through the plan's status word.  The K representatives come from the
// pooling kernel run on K alone beforehand.
// =================================================================================================
constexpr int PO_THREADS = 1024;

__device__ __forceinline__ void role_bar(int id) { asm volatile("bar.sync %0, 512;" ::"r"(id) : "memory"); }

template <int D, int HG>
__global__ void __launch_bounds__(PO_THREADS, 1)
pool_observe_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ kmax,
                    const __nv_bfloat16* __restrict__ kmin, __nv_bfloat16* __restrict__ qmax_out,
                    __nv_bfloat16* __restrict__ qmin_out, float* __restrict__ scores, float* __restrict__ entropy,
                    Shape s, double scale, int nsub, int xcap, int n_items, int* __restrict__ status) {
  extern __shared__ __align__(16) unsigned char po_smem[];
  constexpr int QSTR = D + 1;  // doubles per representative row: the odd stride spreads the 8 rows over the banks
  constexpr int LPR = D / 8;   // 16-byte lanes per row
  constexpr int RS = 512 / LPR;  // row slots of the pooling role
  // layout: lse [HG*4] | epart [HG][16] | xs [HG*4][xcap] | reps [2][8][QSTR] (doubles) | smx, smn [512] uint4 | 4 mbarriers
  double* lse = reinterpret_cast<double*>(po_smem);
  double* epart = lse + HG * 4;
  double* xs = epart + HG * OBS_WARPS;
  double* reps = xs + (size_t)HG * 4 * xcap;
  uint4* smx = reinterpret_cast<uint4*>(reps + 2 * 8 * QSTR);  // every block before this holds an even number of doubles
  uint4* smn = smx + 512;
  const uint32_t bar0 = smem_u32(smn + 512);
  auto FULL = [&](int b) { return bar0 + 8u * b; };
  auto EMPTY = [&](int b) { return bar0 + 16u + 8u * b; };

  // an earlier wait gave up: do nothing (decided for the whole CTA at once, so no warp is left at a barrier)
  if (__syncthreads_or(*reinterpret_cast<volatile int*>(status) != 0)) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int b = 0; b < 2; ++b) {
      mbar_init(FULL(b), 1);
      mbar_init(EMPTY(b), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  auto decode = [&](int n, int& g, int& sub, int& i) {  // longest rows first, as in observe_kernel
    int it = blockIdx.x + n * gridDim.x;
    sub = it % nsub;
    it /= nsub;
    g = it % s.Hkv;
    i = s.C_S - 1 - it / s.Hkv;
  };
  const int n_my = (n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

  if (warp >= 16) {
    // ================= pooling role: query cells of row n into reps[n & 1] =================
    const int ptid = tid - 512, lane16 = ptid % LPR, slot = ptid / LPR;
    constexpr int UNROLL = 8, HB = UNROLL / 2;
    const uint32_t NEG = 0xFF80FF80u, POS = 0x7F807F80u;  // bf16x2 -inf / +inf
    // Two groups of four 16-byte loads leapfrog: while one group is folded in, the other is in flight.  The
    // first two groups of the NEXT cell are issued before the current cell's cross-thread reduction, so the
    // memory pipe does not drain at cell boundaries.
    uint4 va[HB], vb[HB];
    const __nv_bfloat16* p = nullptr;  // this thread's column slice of the current cell's first row
    int L = 0;                         // rows of the current cell (0: a head this sub-group does not have)
    auto locate = [&](int n, int hh, const __nv_bfloat16*& pp, int& LL) {
      int g, sub, i;
      decode(n, g, sub, i);
      const int nh = min(HG, s.G - sub * HG);
      LL = hh < nh ? (int)min((long long)s.L_S, (long long)s.Nq - (long long)i * s.L_S) : 0;
      pp = q + (long long)(g * s.G + sub * HG + (hh < nh ? hh : 0)) * s.qs_h + (long long)i * s.L_S * s.qs_t + lane16 * 8;
    };
    auto load = [&](uint4 (&v)[HB], int row0) {
#pragma unroll
      for (int u = 0; u < HB; ++u) {
        const int row = row0 + u * RS;
        if (row < L) v[u] = ld_stream(p + (long long)row * s.qs_t);
      }
    };
    if (n_my > 0) {
      locate(0, 0, p, L);
      load(va, slot);
      load(vb, slot + HB * RS);
    }
    for (int n = 0; n < n_my; ++n) {
      const int b = n & 1;
      int g, sub, i;
      decode(n, g, sub, i);
      const int h0 = g * s.G + sub * HG, nh = min(HG, s.G - sub * HG);
      double* rb = reps + b * 8 * QSTR;
      for (int hh = 0; hh < HG; ++hh) {
        uint4 mx = make_uint4(NEG, NEG, NEG, NEG), mn = make_uint4(POS, POS, POS, POS);
        auto fold = [&](const uint4 (&v)[HB], int row0) {
#pragma unroll
          for (int u = 0; u < HB; ++u) {
            const int row = row0 + u * RS;
            if (row < L) {
              acc_max(mx, v[u]);
              acc_min(mn, v[u]);
            }
          }
        };
        for (int row0 = slot; row0 < L; row0 += RS * UNROLL) {
          fold(va, row0);
          load(va, row0 + RS * UNROLL);
          fold(vb, row0 + HB * RS);
          load(vb, row0 + RS * UNROLL + HB * RS);
        }
        // next cell: the next head of this row, else the first head of the next row
        if (hh + 1 < HG) {
          locate(n, hh + 1, p, L);
        } else if (n + 1 < n_my) {
          locate(n + 1, 0, p, L);
        } else {
          L = 0;
        }
        load(va, slot);
        load(vb, slot + HB * RS);
        // the row slots of one warp meet through shuffles, the 16 warps through one shared-memory exchange
        // (double-buffered by cell parity, so one barrier per cell is enough)
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) {
          uint4 t;
          t.x = __shfl_xor_sync(0xffffffffu, mx.x, o); t.y = __shfl_xor_sync(0xffffffffu, mx.y, o);
          t.z = __shfl_xor_sync(0xffffffffu, mx.z, o); t.w = __shfl_xor_sync(0xffffffffu, mx.w, o);
          acc_max(mx, t);
          t.x = __shfl_xor_sync(0xffffffffu, mn.x, o); t.y = __shfl_xor_sync(0xffffffffu, mn.y, o);
          t.z = __shfl_xor_sync(0xffffffffu, mn.z, o); t.w = __shfl_xor_sync(0xffffffffu, mn.w, o);
          acc_min(mn, t);
        }
        uint4* ex_max = smx + (hh & 1) * 256;  // [16 warps][LPR] of this parity
        uint4* ex_min = smn + (hh & 1) * 256;
        const int pw = ptid >> 5;
        if (lane < LPR) {
          ex_max[pw * LPR + lane] = mx;
          ex_min[pw * LPR + lane] = mn;
        }
        role_bar(1);
        if (ptid < LPR) {
          if (hh == 0 && n >= 2) mbar_wait(EMPTY(b), ((n >> 1) - 1) & 1, status);  // the observation of row n-2 has let go of reps[b]
          uint4 a = ex_max[ptid], c = ex_min[ptid];
#pragma unroll
          for (int w = 1; w < 16; ++w) {
            acc_max(a, ex_max[w * LPR + ptid]);
            acc_min(c, ex_min[w * LPR + ptid]);
          }
          const uint32_t wa[4] = {a.x, a.y, a.z, a.w}, wc[4] = {c.x, c.y, c.z, c.w};
          double* rmax = rb + (hh * 2 + 0) * QSTR + lane16 * 8;
          double* rmin = rb + (hh * 2 + 1) * QSTR + lane16 * 8;
          if (hh < nh) {
            const long long cell = (long long)(h0 + hh) * s.C_S + i;
            reinterpret_cast<uint4*>(qmax_out + cell * D)[lane16] = a;
            reinterpret_cast<uint4*>(qmin_out + cell * D)[lane16] = c;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              rmax[2 * e] = bf16lo(wa[e]);
              rmax[2 * e + 1] = bf16hi(wa[e]);
              rmin[2 * e] = bf16lo(wc[e]);
              rmin[2 * e + 1] = bf16hi(wc[e]);
            }
          } else {  // rows of heads this sub-group does not have: zero, as observe_kernel's registers are
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              rmax[e] = 0.0;
              rmin[e] = 0.0;
            }
          }
        }
      }
      __threadfence_block();
      role_bar(1);
      if (ptid == 0) mbar_arrive(FULL(b));  // (release) reps[b] holds row n
    }
    return;
  }

  // ================= observation role (warps 0-15): observe_kernel with the query operand in shared memory ========
  const int qrow = lane >> 2, qc = lane & 3;
  constexpr int NSS = D / 32;
  for (int n = 0; n < n_my; ++n) {
    const int b = n & 1;
    int g, sub, i;
    decode(n, g, sub, i);
    const int Ci = causal_blocks(s, i);
    const int h0 = g * s.G + sub * HG;
    const int nh = min(HG, s.G - sub * HG);
    mbar_wait(FULL(b), (n >> 1) & 1, status);  // (acquire) the representatives of row n are in reps[b]
    const double* qsm = reps + b * 8 * QSTR + qrow * QSTR + 8 * qc;

    // ---- phase 1: logits (see observe_kernel) ----
    for (int j0 = warp * 8; j0 < Ci; j0 += OBS_WARPS * 8) {
      const int jbA = min(j0 + (qrow >> 1), Ci - 1), jbB = min(j0 + 4 + (qrow >> 1), Ci - 1);
      const __nv_bfloat16* kbase = ((qrow & 1) ? kmin : kmax) + (long long)g * s.KB_cap * D;
      const __nv_bfloat16* krowA = kbase + (long long)jbA * D;
      const __nv_bfloat16* krowB = kbase + (long long)jbB * D;
      double a0 = 0.0, a1 = 0.0, b0 = 0.0, b1 = 0.0;
#pragma unroll
      for (int ss = 0; ss < NSS; ++ss) {
        const uint4 va = __ldg(reinterpret_cast<const uint4*>(krowA + 8 * (qc + 4 * ss)));
        const uint4 vb = __ldg(reinterpret_cast<const uint4*>(krowB + 8 * (qc + 4 * ss)));
        const double ka[8] = {bf16lo(va.x), bf16hi_cvt(va.x), bf16lo(va.y), bf16hi_cvt(va.y),
                              bf16lo(va.z), bf16hi_cvt(va.z), bf16lo(va.w), bf16hi_cvt(va.w)};
        const double kb[8] = {bf16lo(vb.x), bf16hi_cvt(vb.x), bf16lo(vb.y), bf16hi_cvt(vb.y),
                              bf16lo(vb.z), bf16hi_cvt(vb.z), bf16lo(vb.w), bf16hi_cvt(vb.w)};
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          const double qv = qsm[32 * ss + t];
          asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                       : "+d"(a0), "+d"(a1)
                       : "d"(qv), "d"(ka[t]));
          asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                       : "+d"(b0), "+d"(b1)
                       : "d"(qv), "d"(kb[t]));
        }
      }
      const int hh = qrow >> 1, wq = qrow & 1;
      if (hh < HG) {
        const int jwA = j0 + qc, jwB = j0 + 4 + qc;
        if (jwA < Ci) {
          xs[(hh * 4 + wq * 2 + 0) * xcap + jwA] = scale * a0;
          xs[(hh * 4 + wq * 2 + 1) * xcap + jwA] = scale * a1;
        }
        if (jwB < Ci) {
          xs[(hh * 4 + wq * 2 + 0) * xcap + jwB] = scale * b0;
          xs[(hh * 4 + wq * 2 + 1) * xcap + jwB] = scale * b1;
        }
      }
    }
    role_bar(2);
    if (tid == 0) mbar_arrive(EMPTY(b));  // every observation warp is past its last read of reps[b]

    // ---- phase 2: log-sum-exp of each (head, m) row ----
    for (int p = warp; p < nh * 4; p += OBS_WARPS) {
      const double* x = xs + p * xcap;
      double mx = -INFINITY;
      for (int j = lane; j < Ci; j += 32) mx = fmax(mx, x[j]);
      mx = warp_max_d(mx);
      float sum = 0.f;
      for (int j = lane; j < Ci; j += 32) sum += expf((float)(x[j] - mx));
      sum = warp_sum_f(sum);
      if (lane == 0) lse[p] = mx + (double)logf(sum);
    }
    role_bar(2);

    // ---- phase 3: ln A, scores out, entropy ----
    const double LN2 = 0.693147180559945309417232121458;
    for (int hh = 0; hh < nh; ++hh) {
      const double l0 = lse[hh * 4 + 0], l1 = lse[hh * 4 + 1], l2 = lse[hh * 4 + 2], l3 = lse[hh * 4 + 3];
      float* out = scores + (long long)(h0 + hh) * s.SC + row_offset(s, i);
      double e = 0.0;
      for (int j = tid; j < Ci; j += OBS_THREADS) {
        const double a1 = xs[(hh * 4 + 0) * xcap + j] - l0, a2 = xs[(hh * 4 + 1) * xcap + j] - l1;
        const double a3 = xs[(hh * 4 + 2) * xcap + j] - l2, a4 = xs[(hh * 4 + 3) * xcap + j] - l3;
        const double hi12 = fmax(a1, a2), lo12 = fmin(a1, a2);
        const double hi34 = fmax(a3, a4), lo34 = fmin(a3, a4);
        const double u = hi12 + (double)log1pf(expf((float)(lo12 - hi12)));
        const double w = hi34 + (double)log1pf(expf((float)(lo34 - hi34)));
        double l = fmin(fmax(u, w) - LN2, 0.0);
        const float lf = (float)l;
        out[j] = lf + 0.0f;  // canonical zero
        e -= (double)expf(lf) * l;
      }
      e = warp_sum_d(e);
      if (lane == 0) epart[hh * OBS_WARPS + warp] = e;
    }
    role_bar(2);
    if (tid < nh) {
      double e = 0.0;
      for (int w = 0; w < OBS_WARPS; ++w) e += epart[tid * OBS_WARPS + w];
      entropy[(long long)(h0 + tid) * s.C_S + i] = (float)e;
    }
    role_bar(2);  // xs, lse and epart are free for the next row
  }
}

static size_t pool_observe_smem_bytes(int d, int hg, int xcap) {
  // doubles: lse, epart, xs, reps (an even count each) ; then smx, smn ; then 4 mbarriers
  const size_t doubles = (size_t)hg * 4 + (size_t)hg * OBS_WARPS + (size_t)hg * 4 * xcap + 2 * 8 * (size_t)(d + 1);
  return sizeof(double) * doubles + 2 * 512 * 16 + 4 * 8;
}

template <int D, int HG>
static cudaError_t launch_pool_observe_t(const Shape& s, const __nv_bfloat16* q, const __nv_bfloat16* kmax,
                                         const __nv_bfloat16* kmin, __nv_bfloat16* qmax, __nv_bfloat16* qmin,
                                         double scale, float* scores, float* entropy, int* status, cudaStream_t st) {
  const int nsub = (s.G + HG - 1) / HG;
  const size_t smem = pool_observe_smem_bytes(D, HG, s.C_B);
  cudaError_t e = cudaFuncSetAttribute(pool_observe_kernel<D, HG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const long long n_items = (long long)s.C_S * s.Hkv * nsub;
  const unsigned grid = (unsigned)(n_items < 148 ? n_items : 148);  // one CTA per SM, each walks its share of the rows
  pool_observe_kernel<D, HG><<<grid, PO_THREADS, smem, st>>>(q, kmax, kmin, qmax, qmin, scores, entropy, s, scale, nsub,
                                                            s.C_B, (int)n_items, status);
  return cudaGetLastError();
}

bool pool_observe_shape_supported(const Shape& s) {
  const int hg = observe_pick_hg(s);
  return s.d <= 128 && hg != 0 && pool_observe_smem_bytes(s.d, hg, s.C_B) <= 225 * 1024;
}

cudaError_t launch_pool_observe(const Shape& s, const __nv_bfloat16* q, const __nv_bfloat16* kmax,
                                const __nv_bfloat16* kmin, __nv_bfloat16* qmax, __nv_bfloat16* qmin, double scale,
                                float* scores, float* entropy, int* status, cudaStream_t st) {
  const int hg = observe_pick_hg(s);
#define EI_PO(D_, HG_) return launch_pool_observe_t<D_, HG_>(s, q, kmax, kmin, qmax, qmin, scale, scores, entropy, status, st)
  if (s.d == 128) {
    if (hg == 4) EI_PO(128, 4);
    if (hg == 2) EI_PO(128, 2);
    if (hg == 1) EI_PO(128, 1);
  } else {
    if (hg == 4) EI_PO(64, 4);
    if (hg == 2) EI_PO(64, 2);
    if (hg == 1) EI_PO(64, 1);
  }
#undef EI_PO
  return cudaErrorInvalidValue;
}

// =================================================================================================
// Group-shared planning (optional tail of stage 1b): the "Averaged" aggregation over the G query heads
// of a KV head,  e_g[i] = (1/G) sum_h e_h[i],  lnA_g[i,j] = ln((1/G) sum_h exp(lnA_h[i,j])).
// fp64 arithmetic on the stored fp32 tables, heads added in index order, so the result is a pure
// function of those tables.
// =================================================================================================
__global__ void __launch_bounds__(256) group_aggregate_kernel(Shape s, const float* __restrict__ scores,
                                                              const float* __restrict__ entropy,
                                                              float* __restrict__ g_scores,
                                                              float* __restrict__ g_entropy, const PackedSeq* pk) {
  if (pk != nullptr) {  // a packed batch: blockIdx.y is my sequence
    const PackedSeq& P = pk[blockIdx.y];
    s = P.s;
    scores += P.sc0;
    entropy += P.cell0;
    g_scores += P.lsc0;
    g_entropy += P.lcell0;
  }
  const long long n_sc = (long long)s.Hkv * s.SC, n_e = (long long)s.Hkv * s.C_S;
  const double inv_g = 1.0 / (double)s.G;
  for (long long x = (long long)blockIdx.x * 256 + threadIdx.x; x < n_sc + n_e; x += (long long)gridDim.x * 256) {
    if (x < n_sc) {
      const long long g = x / s.SC, o = x - g * s.SC;
      const float* src = scores + g * s.G * s.SC + o;
      float mx = -INFINITY;
      for (int t = 0; t < s.G; ++t) mx = fmaxf(mx, src[(long long)t * s.SC]);
      float r = mx;
      if (mx != -INFINITY) {
        double sum = 0.0;
        for (int t = 0; t < s.G; ++t) sum += exp((double)src[(long long)t * s.SC] - (double)mx);
        r = (float)((double)mx + log(sum * inv_g));
      }
      g_scores[x] = r;
    } else {
      const long long y = x - n_sc, g = y / s.C_S, i = y - g * s.C_S;
      double acc = 0.0;
      for (int t = 0; t < s.G; ++t) acc += (double)entropy[(g * s.G + t) * s.C_S + i];
      g_entropy[y] = (float)(acc * inv_g);
    }
  }
}

cudaError_t launch_group_aggregate(const Shape& s, const float* scores, const float* entropy, float* g_scores,
                                   float* g_entropy, cudaStream_t st) {
  const long long n = (long long)s.Hkv * (s.SC + s.C_S);
  long long grid = (n + 255) / 256;
  if (grid > 148 * 8) grid = 148 * 8;
  group_aggregate_kernel<<<(unsigned)grid, 256, 0, st>>>(s, scores, entropy, g_scores, g_entropy, nullptr);
  return cudaGetLastError();
}
cudaError_t launch_group_aggregate_packed(const PackedSeq* pk, const PackedSeq* pk_host, int npk, const float* scores,
                                          const float* entropy, float* g_scores, float* g_entropy, cudaStream_t st) {
  long long nmax = 0;
  for (int i = 0; i < npk; ++i) {
    const Shape& s = pk_host[i].s;
    const long long n = (long long)s.Hkv * (s.SC + s.C_S);
    nmax = n > nmax ? n : nmax;
  }
  long long gx = (nmax + 255) / 256;
  if (gx > 148 * 4) gx = 148 * 4;
  group_aggregate_kernel<<<dim3((unsigned)gx, (unsigned)npk), 256, 0, st>>>(pk_host[0].s, scores, entropy, g_scores, g_entropy, pk);
  return cudaGetLastError();
}

// =================================================================================================
// Stage 2 -- head class, multipliers and block counts (Alg. 3), one CTA.
//   rigid[h] = max_i e[h,i] < e_t;   m[h,0] = 1;
//   m[h,i]   = clamp(m[h,i-1] + alpha*(|e_i - e_{i-1}| / max(e_{i-1}, e_t) - delta_t), 1, max_mult)
// in IEEE fp64 with explicitly rounded operations (no contraction) on the stored fp32 table, so
// the result is a pure function of that table.  Block counts use exact integers:
//   M = floor(m*4096 + 0.5),  k(c, b) = min(C_i, max(r, (M*b) >> 24)),  b in 1/4096 block.
// BASE mode: b = base budget.  TOTAL mode: b* = largest b with sum_c k(c,b) <= T, found by
// bisection (each thread keeps its few cells in registers); the R = T - sum k(c,b*) leftover blocks go to the first
// R cells, in increasing c, whose count grows at b*+1.  Offsets are the exclusive scan of k.
//
// The kernel runs in one piece or in its two halves (a.phase): the multipliers alone (A), and the apportionment
// alone (B, C) over a table of multipliers that may cover MORE heads than this plan holds -- the heads of a layer
// sharded over several GPUs, whose tables were gathered: every shard then finds the same b* and the same
// leftover cells for all H_all heads and keeps the counts of its own heads [first_head, first_head + H).
// =================================================================================================
constexpr int BUD_THREADS = 1024;

// (M*b) >> 24 in 32-bit pieces: with b = bh*4096 + bl, floor(M*b / 2^24) = (M*bh + ((M*bl) >> 12)) >> 12
// exactly (M*bh is an integer).  M <= 4096*max_mult and bh <= C_B keep every product below 2^31.
__device__ __forceinline__ int cell_blocks(int M, long long b, int r, int Ci) {
  const int bh = (int)(b >> 12), bl = (int)(b & 4095);
  int raw = (M * bh + ((M * bl) >> 12)) >> 12;
  raw = max(raw, r);
  return min(raw, Ci);
}

// exclusive block scan of one long long per thread; returns the exclusive prefix, total in *tot
__device__ long long block_excl_scan(long long v, long long* warp_sums, long long* tot) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  long long inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    long long t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();  // protect warp_sums reuse
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    long long w = warp_sums[lane];
    long long winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      long long t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    warp_sums[lane] = winc - w;  // exclusive
    if (lane == 31) warp_sums[32] = winc;
  }
  __syncthreads();
  *tot = warp_sums[32];
  return warp_sums[warp] + inc - v;
}

// class and multiplier recurrence of one head, by one warp (Alg. 3).  The division-heavy increments are computed
// lane-parallel; only add / clamp is sequential.  Every lane carries the same running multiplier, so lane t keeps
// the value after step t of its chunk.
__device__ __forceinline__ void head_multipliers(const Shape& s, const BudgetArgs& a, const float* __restrict__ entropy,
                                                 unsigned char* __restrict__ rigid, int* __restrict__ Mfx, int h, int lane,
                                                 int* s_rigid) {
    const float* e = entropy + (long long)h * s.C_S;
    double emax = -INFINITY;
    for (int i = lane; i < s.C_S; i += 32) emax = fmax(emax, (double)e[i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) emax = fmax(emax, __shfl_xor_sync(0xffffffffu, emax, o));
    const bool rg = emax < a.e_t;
    if (lane == 0) {
      rigid[h] = rg ? 1 : 0;
      if (rg && s_rigid != nullptr) atomicAdd(s_rigid, 1);
    }
    int* Mh = Mfx + (long long)h * s.C_S;
    const long long one_bits = __double_as_longlong(1.0), max_bits = __double_as_longlong(a.max_mult);
    double m = 1.0;
    for (int i0 = 0; i0 < s.C_S; i0 += 32) {
      const int i = i0 + lane;
      double inc = 0.0;
      if (!rg && i >= 1 && i < s.C_S) {
        const double prev = (double)e[i - 1], cur = (double)e[i];
        const double den = fmax(prev, a.e_t);
        const double fluct = __ddiv_rn(fabs(__dsub_rn(cur, prev)), den);
        inc = __dmul_rn(a.alpha, __dsub_rn(fluct, a.delta_t));
      }
      double mine = 1.0;
#pragma unroll
      for (int t = 0; t < 32; ++t) {  // fixed trip count: the 32 broadcasts do not depend on the running value
        const double inc_t = __shfl_sync(0xffffffffu, inc, t);
        if (!rg && i0 + t >= 1 && i0 + t < s.C_S) {
          // clamp to [1, max_mult] on the bit patterns: for non-NaN doubles a negative value has a negative
          // pattern and non-negative values order like their patterns, so signed 64-bit compares give the same
          // result as fmax / fmin with far less latency on the sequential chain
          long long vb = __double_as_longlong(__dadd_rn(m, inc_t));
          vb = vb < one_bits ? one_bits : vb;
          vb = vb > max_bits ? max_bits : vb;
          m = __longlong_as_double(vb);
        }
        if (t == lane) mine = m;
      }
      if (i < s.C_S) Mh[i] = (int)floor(__dadd_rn(__dmul_rn(mine, 4096.0), 0.5));
    }
}

// The recurrences of the heads are independent and bound by the fp64 pipe of the SM they run on (a dependent
// add per segment and head): spread over several CTAs, four heads each, they take a quarter of the time they
// take inside the one-CTA budget kernel, which then runs the apportionment alone.
__global__ void __launch_bounds__(128) multipliers_kernel(Shape s, BudgetArgs a, const float* __restrict__ entropy,
                                                          unsigned char* __restrict__ rigid, int* __restrict__ Mfx) {
  const int h = blockIdx.x * 4 + (threadIdx.x >> 5);
  if (h < s.H) head_multipliers(s, a, entropy, rigid, Mfx, h, threadIdx.x & 31, nullptr);
}

__global__ void __launch_bounds__(BUD_THREADS, 1)
budget_kernel(Shape s, BudgetArgs a, const float* __restrict__ entropy, unsigned char* __restrict__ rigid,
              int* __restrict__ Mfx, const int* Mall, int* __restrict__ kblocks, int* __restrict__ offsets,
              Stats* __restrict__ stats, const PackedSeq* pk) {
  if (pk != nullptr) {  // a packed batch: one CTA per sequence, each on its own share of the tables
    const PackedSeq& P = pk[blockIdx.x];
    s = P.ls;
    a.T = P.T;
    a.H_all = s.H;
    entropy += P.lcell0;
    rigid += P.head0;
    Mfx += P.lcell0;
    kblocks += P.lcell0;
    offsets += P.off0;
    stats += P.index;
  }
  __shared__ long long s_warp[33];
  __shared__ int s_rigid, s_mink, s_maxk;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // the apportionment runs over the cells of all a.H_all heads; mine are [cell_lo, cell_hi)
  const int cells = a.H_all * s.C_S;
  const int cell_lo = a.first_head * s.C_S, cell_hi = cell_lo + (int)s.cells;
  if (tid == 0) {
    s_rigid = 0;
    s_mink = 0x7fffffff;
    s_maxk = 0;
  }
  __syncthreads();
  if (a.phase == EI_BUDGET_PHASE_APPORTION) {  // the classes were made by an earlier launch: count them for the statistics
    for (int h = tid; h < s.H; h += BUD_THREADS)
      if (rigid[h]) atomicAdd(&s_rigid, 1);
  }

  // ---- A: class + multiplier recurrence, one warp per head -------------------------------------------
  for (int h = warp; h < s.H && a.phase != EI_BUDGET_PHASE_APPORTION; h += BUD_THREADS / 32)
    head_multipliers(s, a, entropy, rigid, Mfx, h, lane, &s_rigid);
  __syncthreads();
  if (a.phase == EI_BUDGET_PHASE_MULTIPLIERS) return;  // (block-uniform)
  const int* Mt = a.phase == EI_BUDGET_PHASE_APPORTION ? Mall : Mfx;  // the table the apportionment runs over

  // ---- B: base budget: plain bisection, every thread evaluating its own few cells per round ------
  const int cpt = (cells + BUD_THREADS - 1) / BUD_THREADS;
  const int c0 = tid * cpt, c1 = min(cells, c0 + cpt);
  const int i_first = c0 < cells ? c0 % s.C_S : 0;
  constexpr int CACHE = 8;  // cells per thread kept in registers (covers 8192 cells)
  int Mreg[CACHE], Creg[CACHE];
#pragma unroll
  for (int t = 0; t < CACHE; ++t) {
    const int c = c0 + t;
    Mreg[t] = (c < c1) ? Mt[c] : 0;
    Creg[t] = (c < c1) ? causal_blocks(s, (i_first + t) % s.C_S) : 0;
  }
  __shared__ int s_acc[3];  // round r of the search adds into s_acc[r % 3]: one barrier per round (see below)
  if (tid < 3) s_acc[tid] = 0;
  __syncthreads();
  int round = 0;
  // sum over all cells of k(c, b): every thread evaluates its own cells (from registers when they fit),
  // 32-bit partial sums (a thread's cells hold < 2^31 blocks; the total was checked to fit int32)
  auto block_total = [&](long long bcand) -> long long {
    const int bh = (int)(bcand >> 12), bl = (int)(bcand & 4095);
    auto kc = [&](int M, int Ci) {
      int raw = (M * bh + ((M * bl) >> 12)) >> 12;
      return min(max(raw, s.r), Ci);
    };
    int t = 0;
    if (cpt <= 4) {
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (c0 + u < c1) t += kc(Mreg[u], Creg[u]);
    } else if (cpt <= CACHE) {
#pragma unroll
      for (int u = 0; u < CACHE; ++u)
        if (c0 + u < c1) t += kc(Mreg[u], Creg[u]);
    } else {
      for (int c = c0, i = i_first; c < c1; ++c, i = (i + 1 == s.C_S ? 0 : i + 1)) t += kc(Mt[c], causal_blocks(s, i));
    }
    // one warp-wide sum, one shared-memory add per warp, one barrier: the accumulator of round r + 2 was last read
    // before the barrier of round r + 1, so thread 0 may clear it once this round's barrier has passed
    t = __reduce_add_sync(0xffffffffu, t);
    int* acc = &s_acc[round % 3];
    if (lane == 0) atomicAdd(acc, t);
    __syncthreads();
    const int v = *reinterpret_cast<volatile int*>(acc);
    if (tid == 0) s_acc[(round + 2) % 3] = 0;
    ++round;
    return (long long)v;  // the same value in every thread
  };
  long long bstar;
  if (a.mode == EI_BUDGET_BASE_TOKENS) {
    bstar = a.b_fx_base;
  } else {
    long long lo = 0, hi = 4096LL * s.C_B;  // total(0) = cells*r <= T was checked on the host
    if (block_total(hi) <= a.T) {
      lo = hi;
    } else {
      while (hi - lo > 1) {  // invariant: total(lo) <= T < total(hi)
        const long long mid = lo + (hi - lo) / 2;
        if (block_total(mid) <= a.T)
          lo = mid;
        else
          hi = mid;
      }
    }
    bstar = lo;
  }

  // ---- C: counts, leftover distribution, offsets ---------------------------------------------------
  long long R = 0, total1;
  int kmin = 0x7fffffff, kmax = 0;
  if (cpt <= CACHE) {
    // every thread's cells are in registers: counts once, one scan for both the block sum (high word) and the
    // number of cells that grow at b* + 1 (low word), one scan for the offsets
    int kreg[CACHE];
    unsigned grow = 0;
    long long packed = 0;
#pragma unroll
    for (int u = 0; u < CACHE; ++u) {
      kreg[u] = 0;
      if (c0 + u < c1) {
        const int k0 = cell_blocks(Mreg[u], bstar, s.r, Creg[u]);
        kreg[u] = k0;
        packed += (long long)k0 << 32;
        if (a.mode == EI_BUDGET_TOTAL_FRACTION && cell_blocks(Mreg[u], bstar + 1, s.r, Creg[u]) > k0) {
          grow |= 1u << u;
          packed += 1;
        }
      }
    }
    long long tot;
    const long long pre = block_excl_scan(packed, s_warp, &tot);
    if (a.mode == EI_BUDGET_TOTAL_FRACTION) R = a.T - (tot >> 32);
    long long grow_before = pre & 0xffffffffLL;
    long long my_sum = 0;
#pragma unroll
    for (int u = 0; u < CACHE; ++u) {
      const int c = c0 + u;
      if (c < c1) {
        if ((grow >> u) & 1u) {
          if (grow_before < R) kreg[u] += 1;
          grow_before += 1;
        }
        if (c >= cell_lo && c < cell_hi) {
          kblocks[c - cell_lo] = kreg[u];
          my_sum += kreg[u];
          kmin = min(kmin, kreg[u]);
          kmax = max(kmax, kreg[u]);
        } else {
          kreg[u] = 0;  // not mine: no share of the offsets
        }
      }
    }
    long long off = block_excl_scan(my_sum, s_warp, &total1);
#pragma unroll
    for (int u = 0; u < CACHE; ++u) {
      const int c = c0 + u;
      if (c < c1 && c >= cell_lo && c < cell_hi) {
        offsets[c - cell_lo] = (int)off;
        off += kreg[u];
      }
    }
  } else {
    long long base_sum = 0, grow_cnt = 0;
    for (int c = c0, i = i_first; c < c1; ++c, i = (i + 1 == s.C_S ? 0 : i + 1)) {
      const int Ci = causal_blocks(s, i);
      const long long k0 = cell_blocks(Mt[c], bstar, s.r, Ci);
      base_sum += k0;
      if (a.mode == EI_BUDGET_TOTAL_FRACTION) grow_cnt += cell_blocks(Mt[c], bstar + 1, s.r, Ci) > k0;
    }
    long long total0, dummy;
    block_excl_scan(base_sum, s_warp, &total0);
    if (a.mode == EI_BUDGET_TOTAL_FRACTION) R = a.T - total0;
    long long grow_before = block_excl_scan(grow_cnt, s_warp, &dummy);
    long long my_sum = 0;
    for (int c = c0, i = i_first; c < c1; ++c, i = (i + 1 == s.C_S ? 0 : i + 1)) {
      const int Ci = causal_blocks(s, i);
      long long kc = cell_blocks(Mt[c], bstar, s.r, Ci);
      if (a.mode == EI_BUDGET_TOTAL_FRACTION && cell_blocks(Mt[c], bstar + 1, s.r, Ci) > kc) {
        if (grow_before < R) kc += 1;
        grow_before += 1;
      }
      if (c >= cell_lo && c < cell_hi) {
        kblocks[c - cell_lo] = (int)kc;
        my_sum += kc;
        kmin = min(kmin, (int)kc);
        kmax = max(kmax, (int)kc);
      }
    }
    long long off = block_excl_scan(my_sum, s_warp, &total1);
    for (int c = max(c0, cell_lo); c < min(c1, cell_hi); ++c) {
      offsets[c - cell_lo] = (int)off;
      off += kblocks[c - cell_lo];
    }
  }
  if (kmax > 0) {
    atomicMin(&s_mink, kmin);
    atomicMax(&s_maxk, kmax);
  }
  __syncthreads();
  if (tid == 0) {
    offsets[cell_hi - cell_lo] = (int)total1;
    stats->total = total1;
    stats->rigid_heads = s_rigid;
    stats->b_star = bstar;
    stats->leftover = R;
    stats->min_k = s_mink;
    stats->max_k = s_maxk;
    stats->pv_skipped = 0;  // stage 4 counts into it
    stats->reserved1 = 0;
  }
}

cudaError_t launch_budget(const Shape& s, const BudgetArgs& a, const float* entropy, unsigned char* rigid,
                          int* Mfx, const int* Mall, int* kblocks, int* offsets, Stats* stats, cudaStream_t st) {
  if (a.phase != EI_BUDGET_PHASE_APPORTION && s.H >= 8) {  // the recurrences on their own, over several SMs
    multipliers_kernel<<<(s.H + 3) / 4, 128, 0, st>>>(s, a, entropy, rigid, Mfx);
    if (a.phase == EI_BUDGET_PHASE_MULTIPLIERS) return cudaGetLastError();
    BudgetArgs b = a;
    b.phase = EI_BUDGET_PHASE_APPORTION;
    budget_kernel<<<1, BUD_THREADS, 0, st>>>(s, b, entropy, rigid, Mfx, Mfx, kblocks, offsets, stats, nullptr);
    return cudaGetLastError();
  }
  budget_kernel<<<1, BUD_THREADS, 0, st>>>(s, a, entropy, rigid, Mfx, Mall, kblocks, offsets, stats, nullptr);
  return cudaGetLastError();
}

cudaError_t launch_budget_packed(const PackedSeq* pk, int npk, const BudgetArgs& a, const float* entropy,
                                 unsigned char* rigid, int* Mfx, int* kblocks, int* offsets, Stats* stats, cudaStream_t st) {
  budget_kernel<<<npk, BUD_THREADS, 0, st>>>(Shape{}, a, entropy, rigid, Mfx, nullptr, kblocks, offsets, stats, pk);
  return cudaGetLastError();
}

// =================================================================================================
// Stage 3 -- block selection (Eq. t_topk; criticality = ln A_obs).  One warp per (head, segment)
// cell.  Candidates are the non-diagonal causal blocks j < r*i; the warp finds the score of the
// (k - r)-th largest by an 8-bit-digit radix select over order-preserving 32-bit keys (shared
// histogram), then walks the row in index order taking every key above the threshold and the
// lowest-index keys equal to it, which makes ties go to the lower block index and leaves the
// list ascending.  The r diagonal blocks are appended.
// =================================================================================================
constexpr int SEL_WARPS = 4;

__device__ __forceinline__ uint32_t order_key(float f) {
  f += 0.0f;  // -0 -> +0
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__global__ void __launch_bounds__(SEL_WARPS * 32)
select_kernel(Shape s, const float* __restrict__ scores, const int* __restrict__ kblocks,
              const int* __restrict__ offsets, int* __restrict__ indices, int* __restrict__ items, int pairs_per_seg,
              const PackedSeq* pk, int npk) {
  __shared__ int hist[SEL_WARPS][256];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int bid = blockIdx.x;
  if (pk != nullptr) {  // a packed batch: my sequence's shape, my CTA's number within it, its share of the tables
    const PackedSeq& P = pk[packed_find(pk, npk, bid, &PackedSeq::w_sel)];
    s = P.ls;
    bid -= P.w_sel;
    scores += P.lsc0;
    kblocks += P.lcell0;
    offsets += P.off0;
    indices += P.idx0;
    if (items != nullptr) items += P.lcell0 * pairs_per_seg * 8;
  }
  const long long c = (long long)bid * SEL_WARPS + warp;
  if (c >= s.cells) return;
  const int h = (int)(c / s.C_S), i = (int)(c % s.C_S);
  const float* row = scores + (long long)h * s.SC + row_offset(s, i);
  const int ncand = s.c0 + s.r * i;  // blocks before the segment's own rows
  const int k = kblocks[c];
  int* out = indices + offsets[c];
  const int nd = causal_blocks(s, i) - ncand;  // diagonal blocks: r, fewer in a short last segment
  int want = k - nd;
  want = want < 0 ? 0 : (want > ncand ? ncand : want);
  int* hs = hist[warp];

  int written = 0;
  if (want == ncand) {
    for (int j = lane; j < ncand; j += 32) out[j] = j;
    written = ncand;
  } else if (want > 0) {
    uint32_t prefix = 0, mask = 0;
    int remaining = want;  // rank of the threshold among keys matching the prefix (1-based from the top)
    for (int pass = 3; pass >= 0; --pass) {
      const int shift = pass * 8;
      for (int b = lane; b < 256; b += 32) hs[b] = 0;
      __syncwarp();
      for (int j = lane; j < ncand; j += 32) {
        const uint32_t key = order_key(row[j]);
        if ((key & mask) == prefix) atomicAdd(&hs[(key >> shift) & 255], 1);
      }
      __syncwarp();
      // lane l owns bins 255-8l .. 248-8l (descending)
      int cnt[8], lsum = 0;
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        cnt[t] = hs[255 - 8 * lane - t];
        lsum += cnt[t];
      }
      int inc = lsum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      const int excl = inc - lsum;
      const bool mine = (excl < remaining) && (inc >= remaining);
      const unsigned who = __ballot_sync(0xffffffffu, mine);
      const int src = __ffs(who) - 1;
      int digit = 0, above = 0;
      if (mine) {
        int run = excl;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          if (run < remaining && run + cnt[t] >= remaining) {
            digit = 255 - 8 * lane - t;
            above = run;
          }
          run += cnt[t];
        }
      }
      digit = __shfl_sync(0xffffffffu, digit, src);
      above = __shfl_sync(0xffffffffu, above, src);
      remaining -= above;
      prefix |= (uint32_t)digit << shift;
      mask |= 0xFFu << shift;
      __syncwarp();
    }
    // prefix is now the threshold key; take all keys above it and the first `remaining` equal to it
    const uint32_t thr = prefix;
    int eq_seen = 0;
    for (int j0 = 0; j0 < ncand; j0 += 32) {
      const int j = j0 + lane;
      uint32_t key = 0;
      const bool valid = j < ncand;
      if (valid) key = order_key(row[j]);
      const bool eq = valid && key == thr;
      const unsigned eqm = __ballot_sync(0xffffffffu, eq);
      const int eq_rank = eq_seen + __popc(eqm & ((1u << lane) - 1));
      const bool take = valid && (key > thr || (eq && eq_rank < remaining));
      const unsigned tm = __ballot_sync(0xffffffffu, take);
      if (take) out[written + __popc(tm & ((1u << lane) - 1))] = j;
      written += __popc(tm);
      eq_seen += __popc(eqm);
    }
  }
  for (int t = lane; t < nd && t < k; t += 32) out[written + t] = ncand + t;
  if (items != nullptr) {  // the list is complete: the stage-4 records of this cell's tile pairs follow from it
    __syncwarp();
    for (int pr = 0; pr < pairs_per_seg; ++pr)
      attention_item_record(s, i, pr, offsets[c], k, out, items + (c * pairs_per_seg + pr) * 8, lane);
  }
}

cudaError_t launch_select(const Shape& s, const float* scores, const int* kblocks, const int* offsets,
                          int* indices, int* items, cudaStream_t st) {
  const unsigned grid = (unsigned)((s.cells + SEL_WARPS - 1) / SEL_WARPS);
  const int pairs = s.L_S % 256 == 0 ? s.L_S / 256 : 0;  // shapes the tile-pair kernels of stage 4 take
  select_kernel<<<grid, SEL_WARPS * 32, 0, st>>>(s, scores, kblocks, offsets, indices, pairs ? items : nullptr, pairs,
                                                 nullptr, 0);
  return cudaGetLastError();
}

// grid bookkeeping of a packed batch: CTAs of the earlier sequences in each kernel's grid
void packed_fill_work(PackedSeq* pk_host, int npk) {
  int big = 0;
  for (int i = 0; i < npk; ++i)
    if (pk_host[i].s.C_B > pk_host[big].s.C_B) big = i;
  const int nsub = observe_ctas_per_row(pk_host[big].s);
  long long wp = 0, wo = 0, ws = 0, wa = 0;
  for (int i = 0; i < npk; ++i) {
    const Shape& s = pk_host[i].s;
    pk_host[i].w_pool = (int)wp;
    pk_host[i].w_obs = (int)wo;
    pk_host[i].w_sel = (int)ws;
    pk_host[i].w_att = (int)wa;
    wp += s.cells + (long long)s.Hkv * s.C_B;
    wo += (long long)s.C_S * s.Hkv * nsub;
    ws += (pk_host[i].ls.cells + SEL_WARPS - 1) / SEL_WARPS;
    // stage 4: a CTA per tile pair where the two-tile kernels apply, else per 128-row tile
    wa += (long long)s.H * s.C_S * ((s.L_S % 256 == 0 && s.d != 256) ? s.L_S / 256 : s.L_S / 128);
  }
}

cudaError_t launch_select_packed(const PackedSeq* pk, const PackedSeq* pk_host, int npk, const float* scores,
                                 const int* kblocks, const int* offsets, int* indices, int* items, cudaStream_t st) {
  const Shape& s = pk_host[npk - 1].ls;
  const unsigned grid = (unsigned)(pk_host[npk - 1].w_sel + (s.cells + SEL_WARPS - 1) / SEL_WARPS);
  const int pairs = s.L_S % 256 == 0 ? s.L_S / 256 : 0;
  select_kernel<<<grid, SEL_WARPS * 32, 0, st>>>(s, scores, kblocks, offsets, indices, pairs ? items : nullptr, pairs, pk, npk);
  return cudaGetLastError();
}

}  // namespace ei
