// Stage 4 of the EntropyInfer prefill path: causal GQA flash attention over the selected key
// blocks only (the computation counted by Eq. t_spa), hand-written for sm_100a.
//
// One CTA owns one 128-row query tile of one (head, segment) cell and walks that cell's ascending
// block list.  Per key block: K and V tiles arrive by TMA (128-byte swizzle) into shared-memory
// rings, S = Q.K^T and O += P.V run on tcgen05 tensor cores with fp32 accumulators in tensor
// memory, and four softmax warps (one thread per query row) do the online softmax in fp32.
//
//   warp 0-3  softmax: tcgen05.ld S -> scale, causal mask (diagonal blocks only), running max /
//             sum, P = exp2(.) as bf16 back into tensor memory (over S) or shared memory,
//             O rescale when the running max moved by more than 2^8, final O / l -> bf16 -> global
//   warp 4    TMA producer (one elected lane)
//   warp 5    MMA issuer (one elected lane): S(it+1) is issued before P(it).V so the tensor pipe
//             works on the next logits while the softmax warps are busy
//
// Tensor memory: S0 at column 0, S1 at 128, O at 256 (512 columns allocated, one CTA per SM).
// Every mbarrier wait is bounded; on expiry the CTA records EI_ERR_DEVICE_TIMEOUT in the status
// word, drains its own TMA loads, frees its tensor memory and returns.  Once the status word is set
// every later wait (of this and of later CTAs) returns at once, so all threads of a CTA run to the
// common end without taking another path: there is no early exit that only some warps could take.
#include <cuda.h>

#include "ei_internal.cuh"
#include "ei_sm100.cuh"

namespace ei {

// ------------------------------------------------------------------------------------------------
// Kernel
// ------------------------------------------------------------------------------------------------
constexpr int ATT_THREADS = 192;
constexpr int BM = 128;
constexpr uint32_t TM_S0 = 0, TM_S1 = 128, TM_O = 256, TM_COLS = 512;
constexpr float RESCALE_THRESHOLD = 8.0f;  // log2 units

template <int D, int BN, int NS, bool P_SMEM>
struct AttSmem {
  static constexpr int Q_BYTES = BM * D * 2;
  static constexpr int KV_BYTES = BN * D * 2;
  static constexpr int P_BYTES = P_SMEM ? BM * BN * 2 : 0;
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = OFF_Q + Q_BYTES;
  static constexpr int OFF_V = OFF_K + NS * KV_BYTES;
  static constexpr int OFF_P = OFF_V + NS * KV_BYTES;
  static constexpr int OFF_BAR = OFF_P + P_BYTES;
  static constexpr int NBAR = 1 + 4 * NS + 2 + 2 + 1;
  static constexpr int TOTAL = OFF_BAR + NBAR * 8 + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;  // slack for manual 1024-byte alignment
};

template <int D, int BN, int NS, bool P_SMEM>
__global__ void __launch_bounds__(ATT_THREADS, 1)
sparse_attention_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                        const __grid_constant__ CUtensorMap tmv, __nv_bfloat16* __restrict__ out,
                        const int* __restrict__ offsets, const int* __restrict__ indices,
                        int* __restrict__ status, Shape s, float scale_log2, const PackedSeq* pk, int npk) {
  using L = AttSmem<D, BN, NS, P_SMEM>;
  extern __shared__ unsigned char att_smem_raw[];

  const uint32_t raw = smem_u32(att_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gbase = att_smem_raw + (base - raw);
  const uint32_t sQ = base + L::OFF_Q, sK = base + L::OFF_K, sV = base + L::OFF_V, sP = base + L::OFF_P;
  const uint32_t bar0 = base + L::OFF_BAR;
  auto BAR = [&](int i) { return bar0 + 8u * i; };
  const int B_QFULL = 0, B_KFULL = 1, B_VFULL = 1 + NS, B_KEMPTY = 1 + 2 * NS, B_VEMPTY = 1 + 3 * NS,
            B_SFULL = 1 + 4 * NS, B_PFULL = B_SFULL + 2, B_ODONE = B_PFULL + 2;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gbase + L::OFF_BAR + L::NBAR * 8);

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);  // warp-uniform by construction

  // ---- which tile ---------------------------------------------------------------------------------
  const int tiles_per_seg = s.L_S / BM;
  int bid = blockIdx.x;
  int tok0 = 0;  // a packed batch: my sequence starts here in q, k, v, out (the tensor maps span the whole batch)
  if (pk != nullptr) {
    const PackedSeq& P = pk[packed_find(pk, npk, bid, &PackedSeq::w_att)];
    s = P.s;
    bid -= P.w_att;
    tok0 = (int)P.tok0;
    offsets += P.off0;
    indices += P.idx0;
    out += P.tok0 * s.os_t;
  }
  const int qt = bid % tiles_per_seg;
  bid /= tiles_per_seg;
  const int h = bid % s.H;
  const int i = s.C_S - 1 - bid / s.H;  // long lists (late segments) first
  const int g = h / s.G;
  const long long cell = (long long)(h / s.list_div) * s.C_S + i;
  const int q0 = i * s.L_S + qt * BM;
  if (q0 >= s.Nq) return;  // a tile of the short last segment that lies beyond the sequence
  const int off = offsets[cell];
  int n = offsets[cell + 1] - off;
  // blocks lying entirely above the tile's last row are fully masked: the list is ascending, drop the tail
  while (n > 0 && (long long)indices[off + n - 1] * BN > (long long)q0 + s.P + BM - 1) --n;

  if (n == 0) {  // no visible key (only possible with hand-made lists): rows are zero
    if (warp < 4 && q0 + tid < s.Nq) {
      __nv_bfloat16* orow = out + (long long)h * s.os_h + (long long)(q0 + tid) * s.os_t;
      for (int c = 0; c < D / 8; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
    }
    return;
  }

  // ---- set-up ---------------------------------------------------------------------------------------
  if (warp == 4) {
    if (lane == 0) {
      mbar_init(BAR(B_QFULL), 1);
      for (int t = 0; t < NS; ++t) {
        mbar_init(BAR(B_KFULL + t), 1);
        mbar_init(BAR(B_VFULL + t), 1);
        mbar_init(BAR(B_KEMPTY + t), 1);
        mbar_init(BAR(B_VEMPTY + t), 1);
      }
      mbar_init(BAR(B_SFULL), 1);
      mbar_init(BAR(B_SFULL + 1), 1);
      mbar_init(BAR(B_PFULL), 128);
      mbar_init(BAR(B_PFULL + 1), 128);
      mbar_init(BAR(B_ODONE), 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      fence_async_smem();
    }
    __syncwarp();
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  bool ok = true;

  if (warp == 4) {
    // ================= TMA producer (whole warp, elected lane issues) =================
    {
      mbar_expect_tx(BAR(B_QFULL), L::Q_BYTES);
#pragma unroll
      for (int p = 0; p < D / 64; ++p) tma_load_3d(sQ + p * (BM * 128), &tmq, p * 64, tok0 + q0, h, BAR(B_QFULL));
      int issued = 0;
      for (int it = 0; it < n && ok; ++it) {
        const int st = it % NS;
        const uint32_t ph = (it / NS) & 1;
        const int blk = __ldg(indices + off + it);
        ok = mbar_wait(BAR(B_KEMPTY + st), ph ^ 1, status);
        if (!ok) break;
        mbar_expect_tx(BAR(B_KFULL + st), L::KV_BYTES);
#pragma unroll
        for (int p = 0; p < D / 64; ++p)
          tma_load_3d(sK + st * L::KV_BYTES + p * (BN * 128), &tmk, p * 64, tok0 + blk * BN, g, BAR(B_KFULL + st));
        ok = mbar_wait(BAR(B_VEMPTY + st), ph ^ 1, status);
        if (!ok) {  // the K load above is in flight: wait for it before leaving
          mbar_wait_drain(BAR(B_KFULL + st), ph);
          break;
        }
        mbar_expect_tx(BAR(B_VFULL + st), L::KV_BYTES);
#pragma unroll
        for (int p = 0; p < D / 64; ++p)
          tma_load_3d(sV + st * L::KV_BYTES + p * (BN * 128), &tmv, p * 64, tok0 + blk * BN, g, BAR(B_VFULL + st));
        issued = it + 1;
      }
      // Drain: every load this thread issued must have landed before the CTA's shared memory is released.
      mbar_wait_drain(BAR(B_QFULL), 0);
      for (int it = (issued > NS ? issued - NS : 0); it < issued; ++it) {
        mbar_wait_drain(BAR(B_KFULL + it % NS), (it / NS) & 1);
        mbar_wait_drain(BAR(B_VFULL + it % NS), (it / NS) & 1);
      }
    }
  } else if (warp == 5) {
    // ================= MMA issuer (whole warp, elected lane issues) =================
    {
      constexpr uint32_t IDESC_QK = make_idesc(BN, false);
      constexpr uint32_t IDESC_PV = make_idesc(D, true);
      auto issue_qk = [&](int j) -> bool {
        const int st = j % NS;
        if (!mbar_wait(BAR(B_KFULL + st), (j / NS) & 1, status)) return false;
        tc_fence_after();
        const uint32_t d_s = tmem + ((j & 1) ? TM_S1 : TM_S0);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint64_t ad = make_desc(sQ + (ks / 4) * (BM * 128) + (ks % 4) * 32, 16, 1024);
          const uint64_t bd = make_desc(sK + st * L::KV_BYTES + (ks / 4) * (BN * 128) + (ks % 4) * 32, 16, 1024);
          umma_ss(d_s, ad, bd, IDESC_QK, ks > 0 ? 1u : 0u);
        }
        umma_commit(BAR(B_SFULL + (j & 1)));
        umma_commit(BAR(B_KEMPTY + st));
        return true;
      };
      ok = mbar_wait(BAR(B_QFULL), 0, status);
      if (ok) ok = issue_qk(0);
      for (int it = 0; it < n && ok; ++it) {
        const int st = it % NS;
        if (it + 1 < n) {
          ok = issue_qk(it + 1);
          if (!ok) break;
        }
        ok = mbar_wait(BAR(B_PFULL + (it & 1)), (it >> 1) & 1, status);
        if (!ok) break;
        ok = mbar_wait(BAR(B_VFULL + st), (it / NS) & 1, status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_o = tmem + TM_O;
        const uint32_t p_t = tmem + ((it & 1) ? TM_S1 : TM_S0);
#pragma unroll
        for (int ks = 0; ks < BN / 16; ++ks) {
          // V tile: 16 token rows per step (2048 B); N panels of 64 are BN*128 B apart
          const uint64_t bd = make_desc(sV + st * L::KV_BYTES + ks * 2048, BN * 128, 1024);
          const uint32_t acc = (it > 0 || ks > 0) ? 1u : 0u;
          if (P_SMEM) {
            const uint64_t ad = make_desc(sP + (ks / 4) * (BM * 128) + (ks % 4) * 32, 16, 1024);
            umma_ss(d_o, ad, bd, IDESC_PV, acc);
          } else {
            umma_ts(d_o, p_t + ks * 8, bd, IDESC_PV, acc);
          }
        }
        umma_commit(BAR(B_VEMPTY + st));
        umma_commit(BAR(B_ODONE));
      }
    }
  } else {
    // ================= softmax / correction / epilogue (warps 0-3, one row per thread) =================
    const int row = tid;                       // 0..127 == tensor-memory lane
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    const int t_row = q0 + row;                // this thread's query position
    float m_run = -INFINITY, l_run = 0.f;
    for (int it = 0; it < n; ++it) {
      const int buf = it & 1;
      const int blk = __ldg(indices + off + it);
      ok = mbar_wait(BAR(B_SFULL + buf), (it >> 1) & 1, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_s = tmem + lane_base + (buf ? TM_S1 : TM_S0);
      float x[BN];
#pragma unroll
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(t_s + c * 32, r);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) x[c * 32 + e] = __uint_as_float(r[e]) * scale_log2;
      }
      // causal mask: only blocks reaching past the tile's first row need it
      if ((long long)(blk + 1) * BN - 1 > q0 + s.P) {
        const int limit = t_row + s.P - blk * BN;  // key column j is visible iff j <= limit
#pragma unroll
        for (int j = 0; j < BN; ++j)
          if (j > limit) x[j] = -INFINITY;
      }
      float mloc = x[0];
#pragma unroll
      for (int j = 1; j < BN; ++j) mloc = fmaxf(mloc, x[j]);
      const float m_new = fmaxf(m_run, mloc);
      if (it == 0) {
        m_run = m_new;
      } else {
        const bool need = m_new > m_run + RESCALE_THRESHOLD;
        if (__any_sync(0xffffffffu, need)) {
          const float m_use = need ? m_new : m_run;
          const float alpha = need ? fast_ex2(m_run - m_use) : 1.0f;  // m_run = -inf gives 0
          ok = mbar_wait(BAR(B_ODONE), (it - 1) & 1, status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          const uint32_t t_o = tmem + lane_base + TM_O;
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(t_o + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
            tmem_st32(t_o + c * 32, r);
          }
          l_run *= alpha;
          m_run = m_use;
        }
      }
      const float m_safe = (m_run == -INFINITY) ? 0.f : m_run;
      float lsum = 0.f;
#pragma unroll
      for (int j = 0; j < BN; ++j) {
        x[j] = fast_ex2(x[j] - m_safe);
        lsum += x[j];
      }
      l_run += lsum;
      if (P_SMEM && it > 0) {  // the single P buffer is still being read by the previous P.V
        ok = mbar_wait(BAR(B_ODONE), (it - 1) & 1, status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      if (P_SMEM) {
        // K-major, 128-byte swizzled rows: 16-byte chunk index XOR (row & 7) inside each 64-column panel
#pragma unroll
        for (int ch = 0; ch < BN / 8; ++ch) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            __nv_bfloat162 b = __floats2bfloat162_rn(x[ch * 8 + 2 * e], x[ch * 8 + 2 * e + 1]);
            w[e] = *reinterpret_cast<uint32_t*>(&b);
          }
          const uint32_t addr = sP + (ch / 8) * (BM * 128) + row * 128 + (((ch % 8) ^ (row & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
        }
        fence_async_smem();
        tmem_wait_st();  // a rescale may have stored to O
      } else {
#pragma unroll
        for (int c = 0; c < BN / 64; ++c) {
          uint32_t r[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            __nv_bfloat162 b = __floats2bfloat162_rn(x[c * 64 + 2 * e], x[c * 64 + 2 * e + 1]);
            r[e] = *reinterpret_cast<uint32_t*>(&b);
          }
          tmem_st32(t_s + c * 32, r);
        }
        tmem_wait_st();
      }
      tc_fence_before();
      mbar_arrive(BAR(B_PFULL + buf));
    }
    if (ok) {
      ok = mbar_wait(BAR(B_ODONE), (n - 1) & 1, status);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      // rows beyond the sequence (short last segment) were computed on zero-filled Q; they take part in the
      // warp-wide tensor-memory loads below and only their stores are dropped
      const bool in_seq = t_row < s.Nq;
      tc_fence_after();
      const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
      const uint32_t t_o = tmem + lane_base + TM_O;
      __nv_bfloat16* orow = out + (long long)h * s.os_h + (long long)t_row * s.os_t;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(t_o + c * 32, r);
        tmem_wait_ld();
#pragma unroll
        for (int v4 = 0; v4 < 4; ++v4) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(r[v4 * 8 + 2 * e]) * inv,
                                                     __uint_as_float(r[v4 * 8 + 2 * e + 1]) * inv);
            w[e] = *reinterpret_cast<uint32_t*>(&b);
          }
          if (in_seq) reinterpret_cast<uint4*>(orow)[c * 4 + v4] = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
    }
  }

  // ---- teardown -------------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem, TM_COLS);
  }
}

// ------------------------------------------------------------------------------------------------
// Pair kernel: one CTA owns TWO adjacent 128-row query tiles of a cell (segments that are a multiple
// of 256 rows).  Each tile has its own softmax warpgroup, S / O accumulators in tensor memory and
// barriers, so one tile's softmax runs while the tensor pipe works on the other tile:
//
//   warps 0-3  softmax of tile 0      warps 4-7  softmax of tile 1
//   warp  8    TMA producer (K and V tiles share one ring of slots, K_j then V_j)
//   warp  9    MMA issuer:  QK0(0) QK1(0) | PV0(j) QK0(j+1) PV1(j) QK1(j+1) | ...
//
// Tensor memory: S0 at 0, S1 at 128, O0 at 256, O1 at 384; P (bf16) overwrites the low half of
// its tile's S columns, so PV_t(j) is issued before QK_t(j+1) (MMAs of one thread run in order).
// The softmax reads S twice from tensor memory (max pass, then exp pass) in 64-column pieces to
// stay within the register budget of a 320-thread CTA.
// ------------------------------------------------------------------------------------------------
constexpr int ATT2_THREADS = 320;
__host__ __device__ constexpr uint32_t tm2_s(int t) { return 128u * (uint32_t)t; }         // S0 at 0, S1 at 128
__host__ __device__ constexpr uint32_t tm2_o(int t) { return 256u + 128u * (uint32_t)t; }  // O0 at 256, O1 at 384

template <int D, int BN, int NSLOT>
struct Att2Smem {
  static constexpr int Q_BYTES = BM * D * 2;      // one tile
  static constexpr int KV_BYTES = BN * D * 2;
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_RING = 2 * Q_BYTES;
  static constexpr int OFF_BAR = OFF_RING + NSLOT * KV_BYTES;
  static constexpr int NBAR = 2 + 2 * NSLOT + 2 + 2 + 2;
  static constexpr int TOTAL = OFF_BAR + NBAR * 8 + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;
};

template <int D, int BN, int NSLOT>
__global__ void __launch_bounds__(ATT2_THREADS, 1)
sparse_attention_pair_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                             const __grid_constant__ CUtensorMap tmv, __nv_bfloat16* __restrict__ out,
                             const int* __restrict__ offsets, const int* __restrict__ indices,
                             int* __restrict__ status, Shape s, float scale_log2, const PackedSeq* pk, int npk) {
  using L = Att2Smem<D, BN, NSLOT>;
  extern __shared__ unsigned char att_smem_raw[];

  const uint32_t raw = smem_u32(att_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gbase = att_smem_raw + (base - raw);
  const uint32_t sQ = base + L::OFF_Q, sRing = base + L::OFF_RING;
  const uint32_t bar0 = base + L::OFF_BAR;
  auto BAR = [&](int i) { return bar0 + 8u * i; };
  const int B_QFULL = 0, B_FULL = 2, B_EMPTY = 2 + NSLOT, B_SFULL = 2 + 2 * NSLOT, B_PFULL = B_SFULL + 2,
            B_ODONE = B_PFULL + 2;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gbase + L::OFF_BAR + L::NBAR * 8);

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);  // warp-uniform by construction

  const int pairs_per_seg = s.L_S / (2 * BM);
  int bid = blockIdx.x;
  int tok0 = 0;  // a packed batch: my sequence starts here in q, k, v, out (the tensor maps span the whole batch)
  if (pk != nullptr) {
    const PackedSeq& P = pk[packed_find(pk, npk, bid, &PackedSeq::w_att)];
    s = P.s;
    bid -= P.w_att;
    tok0 = (int)P.tok0;
    offsets += P.off0;
    indices += P.idx0;
    out += P.tok0 * s.os_t;
  }
  const int pr = bid % pairs_per_seg;
  bid /= pairs_per_seg;
  const int h = bid % s.H;
  const int i = s.C_S - 1 - bid / s.H;
  const int g = h / s.G;
  const long long cell = (long long)(h / s.list_div) * s.C_S + i;
  const int q0 = i * s.L_S + pr * 2 * BM;
  if (q0 >= s.Nq) return;  // a pair of tiles of the short last segment that lies beyond the sequence
  const int off = offsets[cell];
  const int nlist = offsets[cell + 1] - off;
  // per tile: drop the tail blocks that lie entirely above the tile's last row
  int n1 = nlist;
  while (n1 > 0 && (long long)indices[off + n1 - 1] * BN > (long long)q0 + s.P + 2 * BM - 1) --n1;
  int n0 = n1;
  while (n0 > 0 && (long long)indices[off + n0 - 1] * BN > (long long)q0 + s.P + BM - 1) --n0;

  if (n1 == 0) {
    if (warp < 8 && q0 + tid < s.Nq) {
      __nv_bfloat16* orow = out + (long long)h * s.os_h + (long long)(q0 + tid) * s.os_t;
      for (int c = 0; c < D / 8; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
    }
    return;
  }

  if (warp == 8) {
    if (lane == 0) {
      mbar_init(BAR(B_QFULL), 1);
      mbar_init(BAR(B_QFULL + 1), 1);
      for (int t = 0; t < NSLOT; ++t) {
        mbar_init(BAR(B_FULL + t), 1);
        mbar_init(BAR(B_EMPTY + t), 1);
      }
      for (int t = 0; t < 2; ++t) {
        mbar_init(BAR(B_SFULL + t), 1);
        mbar_init(BAR(B_PFULL + t), 128);
        mbar_init(BAR(B_ODONE + t), 1);
      }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      fence_async_smem();
    }
    __syncwarp();
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  bool ok = true;

  if (warp == 8) {
    // ================= TMA producer (whole warp, elected lane issues) =================
    {
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        mbar_expect_tx(BAR(B_QFULL + t), L::Q_BYTES);
#pragma unroll
        for (int p = 0; p < D / 64; ++p)
          tma_load_3d(sQ + t * L::Q_BYTES + p * (BM * 128), &tmq, p * 64, tok0 + q0 + t * BM, h, BAR(B_QFULL + t));
      }
      int issued = 0;  // ring items issued (K_j is item 2j, V_j is item 2j+1)
      for (int u = 0; u < 2 * n1; ++u) {
        const int slot = u % NSLOT;
        const uint32_t ph = (u / NSLOT) & 1;
        const int blk = __ldg(indices + off + (u >> 1));
        ok = mbar_wait(BAR(B_EMPTY + slot), ph ^ 1, status);
        if (!ok) break;
        mbar_expect_tx(BAR(B_FULL + slot), L::KV_BYTES);
        const CUtensorMap* tm = (u & 1) ? &tmv : &tmk;
#pragma unroll
        for (int p = 0; p < D / 64; ++p)
          tma_load_3d(sRing + slot * L::KV_BYTES + p * (BN * 128), tm, p * 64, tok0 + blk * BN, g, BAR(B_FULL + slot));
        issued = u + 1;
      }
      // Drain: every load issued here must have landed before the CTA's shared memory is released.
      mbar_wait_drain(BAR(B_QFULL), 0);
      mbar_wait_drain(BAR(B_QFULL + 1), 0);
      for (int u = (issued > NSLOT ? issued - NSLOT : 0); u < issued; ++u)
        mbar_wait_drain(BAR(B_FULL + u % NSLOT), (u / NSLOT) & 1);
    }
  } else if (warp == 9) {
    // ================= MMA issuer (whole warp, elected lane issues) =================
    {
      constexpr uint32_t IDESC_QK = make_idesc(BN, false);
      constexpr uint32_t IDESC_PV = make_idesc(D, true);
      auto wait_item = [&](int u) { return mbar_wait(BAR(B_FULL + u % NSLOT), (u / NSLOT) & 1, status); };
      auto issue_qk = [&](int t, int j) {  // S_t = Q_t . K_j^T
        const uint32_t kbase = sRing + ((2 * j) % NSLOT) * L::KV_BYTES;
        const uint32_t qbase = sQ + t * L::Q_BYTES;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint64_t ad = make_desc(qbase + (ks / 4) * (BM * 128) + (ks % 4) * 32, 16, 1024);
          const uint64_t bd = make_desc(kbase + (ks / 4) * (BN * 128) + (ks % 4) * 32, 16, 1024);
          umma_ss(tmem + tm2_s(t), ad, bd, IDESC_QK, ks > 0 ? 1u : 0u);
        }
        umma_commit(BAR(B_SFULL + t));
      };
      auto issue_pv = [&](int t, int j) {  // O_t += P_t . V_j
        const uint32_t vbase = sRing + ((2 * j + 1) % NSLOT) * L::KV_BYTES;
#pragma unroll
        for (int ks = 0; ks < BN / 16; ++ks) {
          const uint64_t bd = make_desc(vbase + ks * 2048, BN * 128, 1024);
          umma_ts(tmem + tm2_o(t), tmem + tm2_s(t) + ks * 8, bd, IDESC_PV, (j > 0 || ks > 0) ? 1u : 0u);
        }
        umma_commit(BAR(B_ODONE + t));
      };
      do {
        if (!(ok = wait_item(0))) break;
        if (n0 > 0) {
          if (!(ok = mbar_wait(BAR(B_QFULL), 0, status))) break;
          tc_fence_after();
          issue_qk(0, 0);
        }
        if (!(ok = mbar_wait(BAR(B_QFULL + 1), 0, status))) break;
        tc_fence_after();
        issue_qk(1, 0);
        umma_commit(BAR(B_EMPTY + 0));  // K_0's slot
        for (int j = 0; j < n1 && ok; ++j) {
          if (j < n0) {
            if (!(ok = mbar_wait(BAR(B_PFULL), j & 1, status))) break;
            if (!(ok = wait_item(2 * j + 1))) break;
            tc_fence_after();
            issue_pv(0, j);
            if (j + 1 < n0) {
              if (!(ok = wait_item(2 * j + 2))) break;
              tc_fence_after();
              issue_qk(0, j + 1);
            }
          }
          if (!(ok = mbar_wait(BAR(B_PFULL + 1), j & 1, status))) break;
          if (!(ok = wait_item(2 * j + 1))) break;
          tc_fence_after();
          issue_pv(1, j);
          umma_commit(BAR(B_EMPTY + (2 * j + 1) % NSLOT));  // V_j's slot
          if (j + 1 < n1) {
            if (!(ok = wait_item(2 * j + 2))) break;
            tc_fence_after();
            issue_qk(1, j + 1);
            umma_commit(BAR(B_EMPTY + (2 * j + 2) % NSLOT));  // K_{j+1}'s slot
          }
        }
      } while (false);
    }
  } else {
    // ================= softmax warpgroups: tile t = warp / 4, one row per thread =================
    const int t = warp >> 2;
    const int nt = t ? n1 : n0;
    const int row = tid & 127;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const int tq0 = q0 + t * BM;
    const int t_row = tq0 + row;
    const uint32_t t_s = tmem + lane_base + tm2_s(t);
    const uint32_t t_o = tmem + lane_base + tm2_o(t);
    float m_run = -INFINITY, l_run = 0.f;  // m_run in raw logit units
    for (int j = 0; j < nt; ++j) {
      const int blk = __ldg(indices + off + j);
      ok = mbar_wait(BAR(B_SFULL + t), j & 1, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const bool masked = (long long)(blk + 1) * BN - 1 > tq0 + s.P;
      const int limit = t_row + s.P - blk * BN;  // key column c is visible iff c <= limit
      // ---- pass 1: row max of the raw logits ----
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
      for (int hf = 0; hf < BN / 64; ++hf) {
        uint32_t r0[32], r1[32];
        tmem_ld32(t_s + hf * 64, r0);
        tmem_ld32(t_s + hf * 64 + 32, r1);
        tmem_wait_ld();
        if (masked) {
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            if (hf * 64 + e > limit) r0[e] = 0xff800000u;
            if (hf * 64 + 32 + e > limit) r1[e] = 0xff800000u;
          }
        }
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
          mx0 = fmax3(mx0, __uint_as_float(r0[e]), __uint_as_float(r1[e]));
          mx1 = fmax3(mx1, __uint_as_float(r0[e + 1]), __uint_as_float(r1[e + 1]));
          mx2 = fmax3(mx2, __uint_as_float(r0[e + 2]), __uint_as_float(r1[e + 2]));
          mx3 = fmax3(mx3, __uint_as_float(r0[e + 3]), __uint_as_float(r1[e + 3]));
        }
      }
      const float mloc = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      const float m_new = fmaxf(m_run, mloc);
      if (j == 0) {
        m_run = m_new;
      } else {
        const bool need = (m_new - m_run) * scale_log2 > RESCALE_THRESHOLD;  // -inf start: inf > 8
        if (__any_sync(0xffffffffu, need)) {
          const float m_use = need ? m_new : m_run;
          const float alpha = need ? fast_ex2((m_run - m_use) * scale_log2) : 1.0f;
          ok = mbar_wait(BAR(B_ODONE + t), (j - 1) & 1, status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(t_o + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
            tmem_st32(t_o + c * 32, r);
          }
          l_run *= alpha;
          m_run = m_use;
        }
      }
      // ---- pass 2: P = exp2((s - m) * scale), row sum, bf16 P into the low half of S ----
      const float mc = (m_run == -INFINITY) ? 0.f : m_run * scale_log2;
      const uint64_t c2 = pack2(scale_log2, scale_log2), nm2 = pack2(-mc, -mc);
      uint64_t sa = 0ull, sb = 0ull;  // packed partial row sums (two independent chains of pairs)
#pragma unroll
      for (int hf = 0; hf < BN / 64; ++hf) {
        uint32_t r0[32], r1[32];
        tmem_ld32(t_s + hf * 64, r0);
        tmem_ld32(t_s + hf * 64 + 32, r1);
        tmem_wait_ld();
        if (masked) {
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            if (hf * 64 + e > limit) r0[e] = 0xff800000u;
            if (hf * 64 + 32 + e > limit) r1[e] = 0xff800000u;
          }
        }
        uint32_t pk[32];
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          float a0, a1, b0, b1;
          unpack2(ffma2(pack2(__uint_as_float(r0[e]), __uint_as_float(r0[e + 1])), c2, nm2), a0, a1);
          unpack2(ffma2(pack2(__uint_as_float(r1[e]), __uint_as_float(r1[e + 1])), c2, nm2), b0, b1);
          a0 = fast_ex2(a0);
          a1 = fast_ex2(a1);
          b0 = fast_ex2(b0);
          b1 = fast_ex2(b1);
          sa = fadd2(sa, pack2(a0, a1));
          sb = fadd2(sb, pack2(b0, b1));
          __nv_bfloat162 pa = __floats2bfloat162_rn(a0, a1);
          __nv_bfloat162 pb = __floats2bfloat162_rn(b0, b1);
          pk[e / 2] = *reinterpret_cast<uint32_t*>(&pa);
          pk[16 + e / 2] = *reinterpret_cast<uint32_t*>(&pb);
        }
        tmem_st32(t_s + hf * 32, pk);  // 64 bf16 = 32 columns
      }
      {
        float s0, s1, s2, s3;
        unpack2(sa, s0, s1);
        unpack2(sb, s2, s3);
        l_run += (s0 + s1) + (s2 + s3);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(BAR(B_PFULL + t));
    }
    if (ok && nt > 0) {
      ok = mbar_wait(BAR(B_ODONE + t), (nt - 1) & 1, status);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      const bool in_seq = t_row < s.Nq;  // rows beyond the sequence join the warp-wide loads, only their stores are dropped
      __nv_bfloat16* orow = out + (long long)h * s.os_h + (long long)t_row * s.os_t;
      if (nt == 0) {
        for (int c = 0; c < D / 8 && in_seq; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
      } else {
        tc_fence_after();
        const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(t_o + c * 32, r);
          tmem_wait_ld();
#pragma unroll
          for (int v4 = 0; v4 < 4; ++v4) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(r[v4 * 8 + 2 * e]) * inv,
                                                       __uint_as_float(r[v4 * 8 + 2 * e + 1]) * inv);
              w[e] = *reinterpret_cast<uint32_t*>(&b);
            }
            if (in_seq) reinterpret_cast<uint4*>(orow)[c * 4 + v4] = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem, TM_COLS);
  }
}

// O[row, 0..COLS) *= alpha for this thread's row (rare: only when the running max moved by more than
// 2^8).  Out of line so that its 32-register staging does not add to the softmax loop's pressure.
template <int COLS>
__device__ __noinline__ void rescale_cols(uint32_t t_o, float alpha) {
  tc_fence_after();
#pragma unroll
  for (int c = 0; c < COLS / 32; ++c) {
    uint32_t o[32];
    tmem_ld32(t_o + c * 32, o);
    tmem_wait_ld();
#pragma unroll
    for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
    tmem_st32(t_o + c * 32, o);
  }
}

// ------------------------------------------------------------------------------------------------
// Split-row pair kernel: as the pair kernel, but every query row is shared by TWO softmax threads,
// each owning half of the key columns of S and half of the O columns.  A thread reads its half row
// from tensor memory once and keeps it in registers for both the max and the exp step; the two
// halves agree on the row maximum through a shared-memory atomic max (a running maximum per row,
// never reset) and a 64-thread named barrier between the two warps that share 32 rows.  Sixteen softmax warps (four per scheduler) hide the
// tensor-memory and special-function latencies that limit the 8-warp version.  P is handed to the
// MMA warp in two parts, so P.V starts on the first half of every thread's columns while the second
// half is still being exponentiated.
//
//   warps 0-7   tile 0: warp w -> rows 32*(w%4).., columns (w/4)*BN/2..
//   warps 8-15  tile 1
//   warp 16     TMA producer          warp 17   MMA issuer
// ------------------------------------------------------------------------------------------------
constexpr int ATT3_THREADS = 576;

template <int D, int BN, int NSLOT>
struct Att3Smem {
  static constexpr int Q_BYTES = BM * D * 2;
  static constexpr int KV_BYTES = BN * D * 2;
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_RING = 2 * Q_BYTES;
  static constexpr int OFF_MX = OFF_RING + NSLOT * KV_BYTES;  // int [2 tiles][128 rows]: running row max (ordered key)
  static constexpr int OFF_SKIP = OFF_MX + 2 * BM * 4;        // int [2 tiles][2]: softmax warps that wrote P = 0 (by block parity)
  static constexpr int OFF_BAR = OFF_SKIP + 16;
  static constexpr int NBAR = 2 + 2 * NSLOT + 2 + 4 + 2;  // q_full[2], ring full/empty, s_full[2], p_full[2 tiles][2 halves], o_done[2]
  static constexpr int TOTAL = OFF_BAR + NBAR * 8 + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;
};

// order-preserving float <-> int map for atomicMax on shared memory
__device__ __forceinline__ int f2ord(float f) {
  const int b = __float_as_int(f);
  return b >= 0 ? b : b ^ 0x7fffffff;
}
__device__ __forceinline__ float ord2f(int k) { return __int_as_float(k >= 0 ? k : k ^ 0x7fffffff); }

__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

template <int D, int BN, int NSLOT>
__global__ void __maxnreg__(96)
sparse_attention_split_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                              const __grid_constant__ CUtensorMap tmv, __nv_bfloat16* __restrict__ out,
                              const int* __restrict__ offsets, const int* __restrict__ indices,
                              int* __restrict__ status, Shape s, float scale_log2, float skip_log2,
                              long long* __restrict__ pv_skipped) {
  using L = Att3Smem<D, BN, NSLOT>;
  constexpr int CH = BN / 2;  // S columns per softmax thread
  static_assert(BN == 128, "the split-row kernel is written for 128-wide key blocks");
  constexpr int OH = D / 2;   // O columns per softmax thread
  extern __shared__ unsigned char att_smem_raw[];

  const uint32_t raw = smem_u32(att_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gbase = att_smem_raw + (base - raw);
  const uint32_t sQ = base + L::OFF_Q, sRing = base + L::OFF_RING;
  int* mxcell = reinterpret_cast<int*>(gbase + L::OFF_MX);
  int* skipcnt = reinterpret_cast<int*>(gbase + L::OFF_SKIP);
  const uint32_t bar0 = base + L::OFF_BAR;
  auto BAR = [&](int i) { return bar0 + 8u * i; };
  const int B_QFULL = 0, B_FULL = 2, B_EMPTY = 2 + NSLOT, B_SFULL = 2 + 2 * NSLOT, B_PFULL = B_SFULL + 2,
            B_ODONE = B_PFULL + 4;  // p_full: index 2*t + part
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gbase + L::OFF_BAR + L::NBAR * 8);

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);

  const int pairs_per_seg = s.L_S / (2 * BM);
  int bid = blockIdx.x;
  const int pr = bid % pairs_per_seg;
  bid /= pairs_per_seg;
  const int h = bid % s.H;
  const int i = s.C_S - 1 - bid / s.H;
  const int g = h / s.G;
  const long long cell = (long long)(h / s.list_div) * s.C_S + i;
  const int q0 = i * s.L_S + pr * 2 * BM;
  if (q0 >= s.Nq) return;  // a pair of tiles of the short last segment that lies beyond the sequence
  // The producer warp initialises the barriers and starts the Q loads (they depend only on the block
  // index) before anyone has read the block list, so the first tiles are in flight during set-up.
  if (warp == 16) {
    if (lane == 0) {
      mbar_init(BAR(B_QFULL), 1);
      mbar_init(BAR(B_QFULL + 1), 1);
      for (int t = 0; t < NSLOT; ++t) {
        mbar_init(BAR(B_FULL + t), 1);
        mbar_init(BAR(B_EMPTY + t), 1);
      }
      for (int t = 0; t < 2; ++t) {
        mbar_init(BAR(B_SFULL + t), 1);
        mbar_init(BAR(B_PFULL + 2 * t), 256);
        mbar_init(BAR(B_PFULL + 2 * t + 1), 256);
        mbar_init(BAR(B_ODONE + t), 1);
      }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      fence_async_smem();
    }
    __syncwarp();
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      mbar_expect_tx(BAR(B_QFULL + t), L::Q_BYTES);
#pragma unroll
      for (int p = 0; p < D / 64; ++p)
        tma_load_3d(sQ + t * L::Q_BYTES + p * (BM * 128), &tmq, p * 64, q0 + t * BM, h, BAR(B_QFULL + t));
    }
  }
  const int off = offsets[cell];
  const int nlist = offsets[cell + 1] - off;
  int n1 = nlist;
  while (n1 > 0 && (long long)indices[off + n1 - 1] * BN > (long long)q0 + s.P + 2 * BM - 1) --n1;
  int n0 = n1;
  while (n0 > 0 && (long long)indices[off + n0 - 1] * BN > (long long)q0 + s.P + BM - 1) --n0;

  if (tid < 2 * BM) mxcell[tid] = f2ord(-INFINITY);
  if (tid < 4) skipcnt[tid] = 0;

  // ring items: K_j is item 2j, V_j is item 2j+1; the first NSLOT need no free-slot wait
  auto load_item = [&](int u, int blk) {
    const int slot = u % NSLOT;
    mbar_expect_tx(BAR(B_FULL + slot), L::KV_BYTES);
    const CUtensorMap* tm = (u & 1) ? &tmv : &tmk;
#pragma unroll
    for (int p = 0; p < D / 64; ++p)
      tma_load_3d(sRing + slot * L::KV_BYTES + p * (BN * 128), tm, p * 64, blk * BN, g, BAR(B_FULL + slot));
  };
  int issued = 0;
  // testing aid (ei_plan_debug_waits): one ring item the producer leaves out, so that a bounded wait runs out
  const int skip_item = warp == 16 ? reinterpret_cast<volatile int*>(status)[2] - 1 : -1;
  if (warp == 16 && n1 > 0) {
    for (int u = 0; u < 2 * n1 && u < NSLOT; ++u) {
      if (u != skip_item) load_item(u, __ldg(indices + off + (u >> 1)));
      issued = u + 1;
    }
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  if (n1 == 0) {  // no visible key (only possible with hand-made lists): rows are zero
    if (tid < 2 * BM && q0 + tid < s.Nq) {
      __nv_bfloat16* orow = out + (long long)h * s.os_h + (long long)(q0 + tid) * s.os_t;
      for (int c = 0; c < D / 8; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
    }
    if (warp == 16) {  // the Q loads are in flight: let them land before the CTA goes away
      mbar_wait_drain(BAR(B_QFULL), 0);
      mbar_wait_drain(BAR(B_QFULL + 1), 0);
    }
    return;
  }
  const uint32_t tmem = *tmem_slot;

  bool ok = true;

  if (warp == 16) {
    // ================= TMA producer (whole warp, elected lane issues) =================
    int blk = (issued < 2 * n1) ? __ldg(indices + off + (issued >> 1)) : 0;
    for (int u = issued; u < 2 * n1; ++u) {
      const int slot = u % NSLOT;
      const uint32_t ph = (u / NSLOT) & 1;
      const int blk_next = ((u & 1) && (u >> 1) + 1 < n1) ? __ldg(indices + off + (u >> 1) + 1) : blk;
      ok = mbar_wait(BAR(B_EMPTY + slot), ph ^ 1, status);
      if (!ok) break;
      if (u != skip_item) load_item(u, blk);
      issued = u + 1;
      blk = blk_next;
    }
    // Drain: every load issued here must have landed before the CTA's shared memory is released.
    mbar_wait_drain(BAR(B_QFULL), 0);
    mbar_wait_drain(BAR(B_QFULL + 1), 0);
    for (int u = (issued > NSLOT ? issued - NSLOT : 0); u < issued; ++u)
      if (u != skip_item) mbar_wait_drain(BAR(B_FULL + u % NSLOT), (u / NSLOT) & 1);
  } else if (warp == 17) {
    // ================= MMA issuer (whole warp, elected lane issues) =================
    constexpr uint32_t IDESC_QK = make_idesc(BN, false);
    constexpr uint32_t IDESC_PV = make_idesc(D, true);
    auto wait_item = [&](int u) { return mbar_wait(BAR(B_FULL + u % NSLOT), (u / NSLOT) & 1, status); };
    auto issue_qk = [&](int t, int j) {  // S_t = Q_t . K_j^T
      const uint32_t kbase = sRing + ((2 * j) % NSLOT) * L::KV_BYTES;
      const uint32_t qbase = sQ + t * L::Q_BYTES;
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const uint64_t ad = make_desc(qbase + (ks / 4) * (BM * 128) + (ks % 4) * 32, 16, 1024);
        const uint64_t bd = make_desc(kbase + (ks / 4) * (BN * 128) + (ks % 4) * 32, 16, 1024);
        umma_ss(tmem + tm2_s(t), ad, bd, IDESC_QK, ks > 0 ? 1u : 0u);
      }
      umma_commit(BAR(B_SFULL + t));
    };
    // O_t += P_t . V_j in two parts: part 0 uses the key groups whose P columns the softmax threads write
    // first (k-steps 0,1 of each column half), part 1 the rest, so P.V starts while exp is still running.
    auto issue_pv = [&](int t, int j, int part) {
      const uint32_t vbase = sRing + ((2 * j + 1) % NSLOT) * L::KV_BYTES;
      constexpr int KS = BN / 16, HALF = KS / 2, QUART = KS / 4;
#pragma unroll
      for (int u = 0; u < HALF; ++u) {
        const int ks = (u / QUART) * HALF + part * QUART + (u % QUART);  // BN=128: part 0 -> {0,1,4,5}, part 1 -> {2,3,6,7}
        const uint64_t bd = make_desc(vbase + ks * 2048, BN * 128, 1024);
        umma_ts(tmem + tm2_o(t), tmem + tm2_s(t) + ks * 8, bd, IDESC_PV, (j > 0 || part > 0 || u > 0) ? 1u : 0u);
      }
      if (part == 1) umma_commit(BAR(B_ODONE + t));
    };
    do {
      if (!(ok = wait_item(0))) break;
      if (n0 > 0) {
        if (!(ok = mbar_wait(BAR(B_QFULL), 0, status))) break;
        tc_fence_after();
        issue_qk(0, 0);
      }
      if (!(ok = mbar_wait(BAR(B_QFULL + 1), 0, status))) break;
      tc_fence_after();
      issue_qk(1, 0);
      umma_commit(BAR(B_EMPTY + 0));  // K_0's slot
      // EI_FLAG_ATTN_SKIP_ZERO_PV: when all eight softmax warps of a tile wrote P = 0 for block j (every warp counts
      // itself in skipcnt ahead of its first arrival), P.V adds exactly nothing and is not issued; the barriers are
      // committed all the same.
      // Block 0 is always issued (it initialises O).  The slot of parity j & 1 is next counted at block j + 2, whose
      // S this warp issues later in program order, so clearing it here is ordered before those counts.
      auto p_is_zero = [&](int t, int j) {
        volatile int* c = skipcnt + 2 * t + (j & 1);
        const bool z = pv_skipped != nullptr && j > 0 && *c == 8;  // only when the caller asked for it
        __syncwarp();
        if (lane == 0) *c = 0;
        return z;
      };
      int n_skipped = 0;
      for (int j = 0; j < n1 && ok; ++j) {
        if (j < n0) {
          if (!(ok = mbar_wait(BAR(B_PFULL), j & 1, status))) break;
          const bool z0 = p_is_zero(0, j);
          if (!(ok = wait_item(2 * j + 1))) break;
          tc_fence_after();
          if (!z0) issue_pv(0, j, 0);
          if (!(ok = mbar_wait(BAR(B_PFULL + 1), j & 1, status))) break;
          tc_fence_after();
          if (!z0) issue_pv(0, j, 1);
          else umma_commit(BAR(B_ODONE + 0));
          n_skipped += z0;
          if (j + 1 < n0) {
            if (!(ok = wait_item(2 * j + 2))) break;
            tc_fence_after();
            issue_qk(0, j + 1);
          }
        }
        if (!(ok = mbar_wait(BAR(B_PFULL + 2), j & 1, status))) break;
        const bool z1 = p_is_zero(1, j);
        if (!(ok = wait_item(2 * j + 1))) break;
        tc_fence_after();
        if (!z1) issue_pv(1, j, 0);
        if (!(ok = mbar_wait(BAR(B_PFULL + 3), j & 1, status))) break;
        tc_fence_after();
        if (!z1) issue_pv(1, j, 1);
        else umma_commit(BAR(B_ODONE + 1));
        n_skipped += z1;
        umma_commit(BAR(B_EMPTY + (2 * j + 1) % NSLOT));  // V_j's slot
        if (j + 1 < n1) {
          if (!(ok = wait_item(2 * j + 2))) break;
          tc_fence_after();
          issue_qk(1, j + 1);
          umma_commit(BAR(B_EMPTY + (2 * j + 2) % NSLOT));  // K_{j+1}'s slot
        }
      }
      if (lane == 0 && n_skipped) atomicAdd(reinterpret_cast<unsigned long long*>(pv_skipped), (unsigned long long)n_skipped);
    } while (false);
  } else {
    // (after a timed-out wait the softmax threads keep going through the motions -- later waits return at once --
    //  so that every thread of a tile reaches the same named barriers and nobody is left waiting)
    // ================= softmax: tile t = warp / 8, column half ch = (warp / 4) % 2, row = 32*(warp%4)+lane ====
    const int t = warp >> 3;
    const int ch = (warp >> 2) & 1;
    const int nt = t ? n1 : n0;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const int tq0 = q0 + t * BM;
    const int t_row = tq0 + row;
    const uint32_t t_s = tmem + lane_base + tm2_s(t) + ch * CH;        // my half of S
    const uint32_t t_p = tmem + lane_base + tm2_s(t) + ch * (CH / 2);  // my half of P (bf16 pairs)
    const uint32_t t_o = tmem + lane_base + tm2_o(t) + ch * OH;        // my half of O
    int* mycell = mxcell + t * BM + row;
    // the two threads of a row sit in warps w and w+4 of the tile: a 64-thread barrier per (tile, row quarter)
    const int pair_bar = 1 + t * 4 + (warp & 3);
    // Only blocks reaching past the tile's first row need the causal mask: a suffix j >= jm of the list.
    int jm = nt;
    while (jm > 0 && (long long)(__ldg(indices + off + jm - 1) + 1) * BN - 1 > tq0 + s.P) --jm;
    float m_ref = -INFINITY, l_run = 0.f;  // m_ref in raw logit units
    for (int j = 0; j < nt; ++j) {
      ok = mbar_wait(BAR(B_SFULL + t), j & 1, status);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      uint32_t r0[32], r1[32];  // my half row (r1 unused when the half is 32 columns wide)
      tmem_ld32(t_s, r0);
      if (CH == 64) tmem_ld32(t_s + 32, r1);
      tmem_wait_ld();
      if (j >= jm) {
        const int limit = t_row + s.P - __ldg(indices + off + j) * BN - ch * CH;  // my column c is visible iff c <= limit
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          if (e > limit) r0[e] = 0xff800000u;
          if (CH == 64 && e + 32 > limit) r1[e] = 0xff800000u;
        }
      }
      float mx0 = __uint_as_float(r0[0]), mx1 = __uint_as_float(r0[1]);
#pragma unroll
      for (int e = 2; e < 32; e += 2) {
        if (e & 2) mx0 = fmax3(mx0, __uint_as_float(r0[e]), __uint_as_float(r0[e + 1]));
        else mx1 = fmax3(mx1, __uint_as_float(r0[e]), __uint_as_float(r0[e + 1]));
      }
      if (CH == 64) {
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          if (e & 2) mx0 = fmax3(mx0, __uint_as_float(r1[e]), __uint_as_float(r1[e + 1]));
          else mx1 = fmax3(mx1, __uint_as_float(r1[e]), __uint_as_float(r1[e + 1]));
        }
      }
      const float lmax = fmaxf(mx0, mx1);  // the largest logit of my half row
      atomicMax(mycell, f2ord(lmax));
      tc_fence_before();            // my S loads are done before the other half may overwrite S with P
      named_bar_sync(pair_bar, 64);   // both halves of every row of this tile have published their max
      const float m_true = ord2f(*reinterpret_cast<volatile int*>(mycell));  // running row max so far
      if (j == 0) {
        m_ref = m_true;
      } else {
        const bool need = (m_true - m_ref) * scale_log2 > RESCALE_THRESHOLD;  // -inf start: inf > 8
        if (__any_sync(0xffffffffu, need)) {
          const float alpha = need ? fast_ex2((m_ref - m_true) * scale_log2) : 1.0f;
          ok = mbar_wait(BAR(B_ODONE + t), (j - 1) & 1, status);
          ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < OH / 8; ++c) {  // eight columns at a time: this path is rare, registers are not
            uint32_t o[8];
            tmem_ld8(t_o + c * 8, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 8; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st8(t_o + c * 8, o);
          }
          l_run *= alpha;
          if (need) m_ref = m_true;
        }
      }
      // P = exp2((s - m) * scale) in place, row sum, bf16 pairs into my half of the P columns
      const float mc = (m_ref == -INFINITY) ? 0.f : m_ref * scale_log2;
      const uint64_t c2 = pack2(scale_log2, scale_log2), nm2 = pack2(-mc, -mc);
      uint64_t sa = 0ull, sb = 0ull;
      auto exp_chunk = [&](uint32_t (&r)[32], int c) {
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
          float a0, a1, b0, b1;
          unpack2(ffma2(pack2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), c2, nm2), a0, a1);
          unpack2(ffma2(pack2(__uint_as_float(r[e + 2]), __uint_as_float(r[e + 3])), c2, nm2), b0, b1);
          a0 = fast_ex2(a0);
          a1 = fast_ex2(a1);
          b0 = fast_ex2(b0);
          b1 = fast_ex2(b1);
          sa = fadd2(sa, pack2(a0, a1));
          sb = fadd2(sb, pack2(b0, b1));
          __nv_bfloat162 pa = __floats2bfloat162_rn(a0, a1);
          __nv_bfloat162 pb = __floats2bfloat162_rn(b0, b1);
          pk[e / 2] = *reinterpret_cast<uint32_t*>(&pa);
          pk[e / 2 + 1] = *reinterpret_cast<uint32_t*>(&pb);
        }
        tmem_st16(t_p + c * 16, pk);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(BAR(B_PFULL + 2 * t + c));
      };
      // A half row whose largest logit lies more than skip_log2 below the reference maximum holds only terms below
      // 2^-skip_log2 of the row's largest: where that is so for all 32 rows of the warp, P is zero and neither the
      // exponentials nor the sums are evaluated (heads whose attention sits on a few keys spend most blocks here).
      // (lmax = -inf, a fully masked half row, qualifies; m_ref = -inf gives NaN and does not.)
      if (__all_sync(0xffffffffu, (lmax - m_ref) * scale_log2 < -skip_log2)) {
        uint32_t zero[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) zero[e] = 0u;
        tmem_st16(t_p, zero);
        tmem_st16(t_p + 16, zero);
        tmem_wait_st();
        tc_fence_before();
        if (lane == 0) atomicAdd(skipcnt + 2 * t + (j & 1), 1);  // ahead of the arrivals: the MMA warp reads it behind them
        mbar_arrive(BAR(B_PFULL + 2 * t));
        mbar_arrive(BAR(B_PFULL + 2 * t + 1));
      } else {
        exp_chunk(r0, 0);
        exp_chunk(r1, 1);
        float s0, s1, s2, s3;
        unpack2(sa, s0, s1);
        unpack2(sb, s2, s3);
        l_run += (s0 + s1) + (s2 + s3);
      }
    }
    // combine the two halves' row sums through the (no longer needed) max cells
    if (nt > 0) {
      named_bar_sync(pair_bar, 64);
      if (ch == 1) *reinterpret_cast<volatile float*>(mycell) = l_run;
      named_bar_sync(pair_bar, 64);
      const float other1 = *reinterpret_cast<volatile float*>(mycell);
      named_bar_sync(pair_bar, 64);
      if (ch == 0) *reinterpret_cast<volatile float*>(mycell) = l_run;
      named_bar_sync(pair_bar, 64);
      const float other0 = *reinterpret_cast<volatile float*>(mycell);
      l_run += ch ? other0 : other1;
    }
    if (ok && nt > 0) {
      ok = mbar_wait(BAR(B_ODONE + t), (nt - 1) & 1, status);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      const bool in_seq = t_row < s.Nq;  // rows beyond the sequence join the warp-wide loads, only their stores are dropped
      __nv_bfloat16* orow = out + (long long)h * s.os_h + (long long)t_row * s.os_t + ch * OH;
      if (nt == 0) {
        for (int c = 0; c < OH / 8 && in_seq; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
      } else {
        tc_fence_after();
        const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
#pragma unroll
        for (int c = 0; c < OH / 32; ++c) {
          uint32_t o[32];
          tmem_ld32(t_o + c * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int v4 = 0; v4 < 4; ++v4) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(o[v4 * 8 + 2 * e]) * inv,
                                                       __uint_as_float(o[v4 * 8 + 2 * e + 1]) * inv);
              w[e] = *reinterpret_cast<uint32_t*>(&b);
            }
            if (in_seq) reinterpret_cast<uint4*>(orow)[c * 4 + v4] = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 16) {
    tc_fence_after();
    tmem_dealloc(tmem, TM_COLS);
  }
}

// ------------------------------------------------------------------------------------------------
// Persistent form of the split-row kernel.  One CTA per SM keeps its barriers, tensor memory and K/V ring
// for the whole launch and takes (head, segment, tile pair) items off a global counter, longest block lists
// first.  The producer warp is also the scheduler: it takes the next item, looks its block list up, and
// publishes a small record (head, first row, list offset, block counts of the two tiles, first masked
// block) in shared memory two items ahead, so that neither the MMA warp nor the softmax warps touch global
// memory to find their work.  Across an item boundary the Q tiles of the next item are loaded as soon as the
// last Q.K^T of the current one has read them, its first Q.K^T runs while the softmax warps still write the
// current item's output, and its first P.V waits until they have read O out of tensor memory.
// ------------------------------------------------------------------------------------------------
template <int D, int BN, int NSLOT>
struct Att4Smem {
  static constexpr int Q_BYTES = BM * D * 2;
  static constexpr int KV_BYTES = BN * D * 2;
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_RING = 2 * Q_BYTES;
  static constexpr int OFF_MX = OFF_RING + NSLOT * KV_BYTES;  // int [2 tiles][128 rows]
  static constexpr int OFF_INFO = OFF_MX + 2 * BM * 4;        // int [2 slots][8]
  static constexpr int OFF_BAR = OFF_INFO + 2 * 8 * 4;
  // q_full[2] q_empty[2] ring full/empty s_full[2] p_full[4] o_done[2] o_free[2] info_full[2] info_empty[2]
  static constexpr int NBAR = 4 + 2 * NSLOT + 2 + 4 + 2 + 2 + 4;
  static constexpr int TOTAL = OFF_BAR + NBAR * 8 + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;
};

template <int D, int BN, int NSLOT>
__global__ void __maxnreg__(96)
sparse_attention_persistent_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                                   const __grid_constant__ CUtensorMap tmv, __nv_bfloat16* __restrict__ out,
                                   const int* __restrict__ offsets, const int* __restrict__ indices,
                                   int* __restrict__ status, int* __restrict__ sched, Shape s, float scale_log2,
                                   float skip_log2, int n_items) {
  using L = Att4Smem<D, BN, NSLOT>;
  constexpr int CH = BN / 2;
  constexpr int OH = D / 2;
  static_assert(BN == 128, "the split-row kernels are written for 128-wide key blocks");
  extern __shared__ unsigned char att_smem_raw[];

  const uint32_t raw = smem_u32(att_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gbase = att_smem_raw + (base - raw);
  const uint32_t sQ = base + L::OFF_Q, sRing = base + L::OFF_RING;
  int* mxcell = reinterpret_cast<int*>(gbase + L::OFF_MX);
  volatile int* info = reinterpret_cast<volatile int*>(gbase + L::OFF_INFO);
  const uint32_t bar0 = base + L::OFF_BAR;
  auto BAR = [&](int i) { return bar0 + 8u * i; };
  const int B_QFULL = 0, B_QEMPTY = 2, B_FULL = 4, B_EMPTY = 4 + NSLOT, B_SFULL = 4 + 2 * NSLOT,
            B_PFULL = B_SFULL + 2, B_ODONE = B_PFULL + 4, B_OFREE = B_ODONE + 2, B_IFULL = B_OFREE + 2,
            B_IEMPTY = B_IFULL + 2;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gbase + L::OFF_BAR + L::NBAR * 8);
  // record layout
  enum { I_VALID = 0, I_H = 1, I_Q0 = 2, I_OFF = 3, I_N0 = 4, I_N1 = 5, I_JM0 = 6, I_JM1 = 7 };

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);

  if (warp == 16) {
    if (lane == 0) {
      for (int t = 0; t < 2; ++t) {
        mbar_init(BAR(B_QFULL + t), 1);
        mbar_init(BAR(B_QEMPTY + t), 1);
        mbar_init(BAR(B_SFULL + t), 1);
        mbar_init(BAR(B_PFULL + 2 * t), 256);
        mbar_init(BAR(B_PFULL + 2 * t + 1), 256);
        mbar_init(BAR(B_ODONE + t), 1);
        mbar_init(BAR(B_OFREE + t), 256);
        mbar_init(BAR(B_IFULL + t), 1);
        mbar_init(BAR(B_IEMPTY + t), 17);  // the MMA warp and the 16 softmax warps
      }
      for (int t = 0; t < NSLOT; ++t) {
        mbar_init(BAR(B_FULL + t), 1);
        mbar_init(BAR(B_EMPTY + t), 1);
      }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      fence_async_smem();
    }
    __syncwarp();
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // an earlier launch gave up: take no work (one answer per warp, whatever the lanes read)
  const bool dead = __any_sync(0xffffffffu, *reinterpret_cast<volatile int*>(status) != 0);

  bool ok = true;
  const int pairs_per_seg = s.L_S / (2 * BM);

  if (warp == 16) {
    // ================= scheduler + TMA producer =================
    int ucount = 0;  // ring items issued so far, over all work items
    int kk = 0;      // records published so far
    int last_q = -1;  // the last item whose Q tiles were loaded
    for (;; ++kk) {
      int item = n_items;
      if (!dead && ok) {
        if (lane == 0) item = atomicAdd(sched, 1);
        item = __shfl_sync(0xffffffffu, item, 0);
      }
      const bool valid = item < n_items;
      int h = 0, q0 = 0, off = 0, n0 = 0, n1 = 0, jm0 = 0, jm1 = 0, g = 0;
      if (valid) {
        int bid = item;
        const int pr = bid % pairs_per_seg;
        bid /= pairs_per_seg;
        h = bid % s.H;
        const int i = s.C_S - 1 - bid / s.H;  // long lists (late segments) first
        g = h / s.G;
        const long long cell = (long long)(h / s.list_div) * s.C_S + i;
        q0 = i * s.L_S + pr * 2 * BM;
        if (q0 < s.Nq) {  // a pair beyond the sequence (short last segment) keeps n0 = n1 = 0 and stores nothing
          off = __ldg(offsets + cell);
          n1 = __ldg(offsets + cell + 1) - off;
          while (n1 > 0 && (long long)__ldg(indices + off + n1 - 1) * BN > (long long)q0 + s.P + 2 * BM - 1) --n1;
          n0 = n1;
          while (n0 > 0 && (long long)__ldg(indices + off + n0 - 1) * BN > (long long)q0 + s.P + BM - 1) --n0;
          jm0 = n0;
          while (jm0 > 0 && (long long)(__ldg(indices + off + jm0 - 1) + 1) * BN - 1 > q0 + s.P) --jm0;
          jm1 = n1;
          while (jm1 > 0 && (long long)(__ldg(indices + off + jm1 - 1) + 1) * BN - 1 > q0 + BM + s.P) --jm1;
        }
      }
      const int slot_i = kk & 1;
      ok = mbar_wait(BAR(B_IEMPTY + slot_i), ((kk >> 1) & 1) ^ 1, status) && ok;  // record of item kk-2 has been read
      if (lane == 0) {
        volatile int* r = info + slot_i * 8;
        r[I_VALID] = (valid && ok) ? 1 : 0;
        r[I_H] = h;
        r[I_Q0] = q0;
        r[I_OFF] = off;
        r[I_N0] = n0;
        r[I_N1] = n1;
        r[I_JM0] = jm0;
        r[I_JM1] = jm1;
        __threadfence_block();
        mbar_arrive(BAR(B_IFULL + slot_i));
      }
      __syncwarp();
      if (!valid || !ok) break;
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        ok = mbar_wait(BAR(B_QEMPTY + t), (kk & 1) ^ 1, status);  // the previous item's Q.K^T_t are done with Q_t
        if (!ok) break;
        mbar_expect_tx(BAR(B_QFULL + t), L::Q_BYTES);
#pragma unroll
        for (int p = 0; p < D / 64; ++p)
          tma_load_3d(sQ + t * L::Q_BYTES + p * (BM * 128), &tmq, p * 64, q0 + t * BM, h, BAR(B_QFULL + t));
      }
      if (!ok) continue;  // publishes an invalid record next round and stops
      last_q = kk;
      int blk = n1 > 0 ? __ldg(indices + off) : 0;
      for (int u = 0; u < 2 * n1; ++u, ++ucount) {
        const int slot = ucount % NSLOT;
        const uint32_t ph = (ucount / NSLOT) & 1;
        const int blk_next = ((u & 1) && (u >> 1) + 1 < n1) ? __ldg(indices + off + (u >> 1) + 1) : blk;
        ok = mbar_wait(BAR(B_EMPTY + slot), ph ^ 1, status);
        if (!ok) break;
        mbar_expect_tx(BAR(B_FULL + slot), L::KV_BYTES);
        const CUtensorMap* tm = (u & 1) ? &tmv : &tmk;
#pragma unroll
        for (int p = 0; p < D / 64; ++p)
          tma_load_3d(sRing + slot * L::KV_BYTES + p * (BN * 128), tm, p * 64, blk * BN, g, BAR(B_FULL + slot));
        blk = blk_next;
      }
    }
    // Drain: every load issued here must have landed before the CTA's shared memory is released.
    if (last_q >= 0) {
      mbar_wait_drain(BAR(B_QFULL), last_q & 1);
      mbar_wait_drain(BAR(B_QFULL + 1), last_q & 1);
    }
    for (int u = (ucount > NSLOT ? ucount - NSLOT : 0); u < ucount; ++u)
      mbar_wait_drain(BAR(B_FULL + u % NSLOT), (u / NSLOT) & 1);
  } else if (warp == 17) {
    // ================= MMA issuer =================
    constexpr uint32_t IDESC_QK = make_idesc(BN, false);
    constexpr uint32_t IDESC_PV = make_idesc(D, true);
    int ubase = 0;        // ring index of this item's K_0
    int itc[2] = {0, 0};  // iterations issued per tile over all items (parity of p_full)
    auto wait_ring = [&](int u) { return mbar_wait(BAR(B_FULL + u % NSLOT), (u / NSLOT) & 1, status); };
    for (int kk = 0;; ++kk) {
      const int slot_i = kk & 1;
      ok = mbar_wait(BAR(B_IFULL + slot_i), (kk >> 1) & 1, status);
      ok = __all_sync(0xffffffffu, ok);
      const volatile int* r = info + slot_i * 8;
      const int valid = ok ? r[I_VALID] : 0, n0 = r[I_N0], n1 = r[I_N1];
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_IEMPTY + slot_i));
      if (!valid) break;
      const int nn[2] = {n0, n1};
      auto issue_qk = [&](int t, int j) {  // S_t = Q_t . K_j^T ; the item's last one also releases Q_t
        const uint32_t kbase = sRing + ((ubase + 2 * j) % NSLOT) * L::KV_BYTES;
        const uint32_t qbase = sQ + t * L::Q_BYTES;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint64_t ad = make_desc(qbase + (ks / 4) * (BM * 128) + (ks % 4) * 32, 16, 1024);
          const uint64_t bd = make_desc(kbase + (ks / 4) * (BN * 128) + (ks % 4) * 32, 16, 1024);
          umma_ss(tmem + tm2_s(t), ad, bd, IDESC_QK, ks > 0 ? 1u : 0u);
        }
        umma_commit(BAR(B_SFULL + t));
        if (j == nn[t] - 1) umma_commit(BAR(B_QEMPTY + t));
      };
      auto issue_pv = [&](int t, int j, int part) {
        const uint32_t vbase = sRing + ((ubase + 2 * j + 1) % NSLOT) * L::KV_BYTES;
        constexpr int KS = BN / 16, HALF = KS / 2, QUART = KS / 4;
#pragma unroll
        for (int u = 0; u < HALF; ++u) {
          const int ks = (u / QUART) * HALF + part * QUART + (u % QUART);
          const uint64_t bd = make_desc(vbase + ks * 2048, BN * 128, 1024);
          umma_ts(tmem + tm2_o(t), tmem + tm2_s(t) + ks * 8, bd, IDESC_PV, (j > 0 || part > 0 || u > 0) ? 1u : 0u);
        }
        if (part == 1) umma_commit(BAR(B_ODONE + t));
      };
      do {
        // Q_t is free for the next item once this item's Q.K^T_t are done; a tile without blocks frees it after
        // the load has landed (the barrier below) so that a load in flight is never overwritten
        if (n0 == 0) {
          if (!(ok = mbar_wait(BAR(B_QFULL), kk & 1, status))) break;
          umma_commit(BAR(B_QEMPTY));
        }
        if (n1 == 0) {
          if (!(ok = mbar_wait(BAR(B_QFULL + 1), kk & 1, status))) break;
          umma_commit(BAR(B_QEMPTY + 1));
          break;
        }
        if (!(ok = wait_ring(ubase))) break;
        if (n0 > 0) {
          if (!(ok = mbar_wait(BAR(B_QFULL), kk & 1, status))) break;
          tc_fence_after();
          issue_qk(0, 0);
        }
        if (!(ok = mbar_wait(BAR(B_QFULL + 1), kk & 1, status))) break;
        tc_fence_after();
        issue_qk(1, 0);
        umma_commit(BAR(B_EMPTY + ubase % NSLOT));  // K_0's slot
        for (int j = 0; j < n1 && ok; ++j) {
          if (j < n0) {
            if (!(ok = mbar_wait(BAR(B_PFULL), itc[0] & 1, status))) break;
            if (!(ok = wait_ring(ubase + 2 * j + 1))) break;
            if (j == 0 && !(ok = mbar_wait(BAR(B_OFREE), (kk & 1) ^ 1, status))) break;  // the previous O_0 has been read
            tc_fence_after();
            issue_pv(0, j, 0);
            if (!(ok = mbar_wait(BAR(B_PFULL + 1), itc[0] & 1, status))) break;
            tc_fence_after();
            issue_pv(0, j, 1);
            ++itc[0];
            if (j + 1 < n0) {
              if (!(ok = wait_ring(ubase + 2 * j + 2))) break;
              tc_fence_after();
              issue_qk(0, j + 1);
            }
          }
          if (!(ok = mbar_wait(BAR(B_PFULL + 2), itc[1] & 1, status))) break;
          if (!(ok = wait_ring(ubase + 2 * j + 1))) break;
          if (j == 0 && !(ok = mbar_wait(BAR(B_OFREE + 1), (kk & 1) ^ 1, status))) break;
          tc_fence_after();
          issue_pv(1, j, 0);
          if (!(ok = mbar_wait(BAR(B_PFULL + 3), itc[1] & 1, status))) break;
          tc_fence_after();
          issue_pv(1, j, 1);
          ++itc[1];
          umma_commit(BAR(B_EMPTY + (ubase + 2 * j + 1) % NSLOT));  // V_j's slot
          if (j + 1 < n1) {
            if (!(ok = wait_ring(ubase + 2 * j + 2))) break;
            tc_fence_after();
            issue_qk(1, j + 1);
            umma_commit(BAR(B_EMPTY + (ubase + 2 * j + 2) % NSLOT));  // K_{j+1}'s slot
          }
        }
      } while (false);
      if (!ok) break;
      ubase += 2 * n1;
    }
  } else {
    // ================= softmax: tile t = warp / 8, column half ch = (warp / 4) % 2, row = 32*(warp%4)+lane ====
    // (after a timed-out wait the threads keep going through the motions -- later waits return at once -- so that
    //  both warps of a row quarter reach the same named barriers)
    const int t = warp >> 3;
    const int ch = (warp >> 2) & 1;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t t_s = tmem + lane_base + tm2_s(t) + ch * CH;
    const uint32_t t_p = tmem + lane_base + tm2_s(t) + ch * (CH / 2);
    const uint32_t t_o = tmem + lane_base + tm2_o(t) + ch * OH;
    int* mycell = mxcell + t * BM + row;
    const int pair_bar = 1 + t * 4 + (warp & 3);
    int itc = 0;  // iterations of my tile over all items (parity of s_full / o_done)
    for (int kk = 0;; ++kk) {
      const int slot_i = kk & 1;
      ok = mbar_wait(BAR(B_IFULL + slot_i), (kk >> 1) & 1, status);
      ok = __all_sync(0xffffffffu, ok);
      const volatile int* r = info + slot_i * 8;
      const int valid = ok ? r[I_VALID] : 0, h = r[I_H], q0 = r[I_Q0], off = r[I_OFF];
      const int nt = t ? r[I_N1] : r[I_N0];
      const int jm = t ? r[I_JM1] : r[I_JM0];
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_IEMPTY + slot_i));
      if (!valid) break;
      const int tq0 = q0 + t * BM;
      const int t_row = tq0 + row;
      if (ch == 0) *mycell = f2ord(-INFINITY);
      named_bar_sync(pair_bar, 64);
      float m_ref = -INFINITY, l_run = 0.f;
      for (int j = 0; j < nt; ++j, ++itc) {
        ok = mbar_wait(BAR(B_SFULL + t), itc & 1, status);
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();
        uint32_t r0[32], r1[32];
        tmem_ld32(t_s, r0);
        tmem_ld32(t_s + 32, r1);
        tmem_wait_ld();
        if (j >= jm) {
          const int limit = t_row + s.P - __ldg(indices + off + j) * BN - ch * CH;  // my column c is visible iff c <= limit
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            if (e > limit) r0[e] = 0xff800000u;
            if (e + 32 > limit) r1[e] = 0xff800000u;
          }
        }
        float mx0 = __uint_as_float(r0[0]), mx1 = __uint_as_float(r0[1]);
#pragma unroll
        for (int e = 2; e < 32; e += 2) {
          if (e & 2) mx0 = fmax3(mx0, __uint_as_float(r0[e]), __uint_as_float(r0[e + 1]));
          else mx1 = fmax3(mx1, __uint_as_float(r0[e]), __uint_as_float(r0[e + 1]));
        }
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          if (e & 2) mx0 = fmax3(mx0, __uint_as_float(r1[e]), __uint_as_float(r1[e + 1]));
          else mx1 = fmax3(mx1, __uint_as_float(r1[e]), __uint_as_float(r1[e + 1]));
        }
        const float lmax = fmaxf(mx0, mx1);  // the largest logit of my half row
      atomicMax(mycell, f2ord(lmax));
        tc_fence_before();
        named_bar_sync(pair_bar, 64);
        const float m_true = ord2f(*reinterpret_cast<volatile int*>(mycell));
        if (j == 0) {
          m_ref = m_true;
        } else {
          const bool need = (m_true - m_ref) * scale_log2 > RESCALE_THRESHOLD;
          if (__any_sync(0xffffffffu, need)) {
            const float alpha = need ? fast_ex2((m_ref - m_true) * scale_log2) : 1.0f;
            ok = mbar_wait(BAR(B_ODONE + t), (itc - 1) & 1, status);
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();
#pragma unroll 1
            for (int c = 0; c < OH / 8; ++c) {
              uint32_t o[8];
              tmem_ld8(t_o + c * 8, o);
              tmem_wait_ld();
#pragma unroll
              for (int e = 0; e < 8; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
              tmem_st8(t_o + c * 8, o);
            }
            l_run *= alpha;
            if (need) m_ref = m_true;
          }
        }
        const float mc = (m_ref == -INFINITY) ? 0.f : m_ref * scale_log2;
        const uint64_t c2 = pack2(scale_log2, scale_log2), nm2 = pack2(-mc, -mc);
        uint64_t sa = 0ull, sb = 0ull;
        auto exp_chunk = [&](uint32_t (&rr)[32], int c) {
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            float a0, a1, b0, b1;
            unpack2(ffma2(pack2(__uint_as_float(rr[e]), __uint_as_float(rr[e + 1])), c2, nm2), a0, a1);
            unpack2(ffma2(pack2(__uint_as_float(rr[e + 2]), __uint_as_float(rr[e + 3])), c2, nm2), b0, b1);
            a0 = fast_ex2(a0);
            a1 = fast_ex2(a1);
            b0 = fast_ex2(b0);
            b1 = fast_ex2(b1);
            sa = fadd2(sa, pack2(a0, a1));
            sb = fadd2(sb, pack2(b0, b1));
            __nv_bfloat162 pa = __floats2bfloat162_rn(a0, a1);
            __nv_bfloat162 pb = __floats2bfloat162_rn(b0, b1);
            pk[e / 2] = *reinterpret_cast<uint32_t*>(&pa);
            pk[e / 2 + 1] = *reinterpret_cast<uint32_t*>(&pb);
          }
          tmem_st16(t_p + c * 16, pk);
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(BAR(B_PFULL + 2 * t + c));
        };
        // negligible half rows: see the per-CTA kernel
        if (__all_sync(0xffffffffu, (lmax - m_ref) * scale_log2 < -skip_log2)) {
          uint32_t zero[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) zero[e] = 0u;
          tmem_st16(t_p, zero);
          tmem_st16(t_p + 16, zero);
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(BAR(B_PFULL + 2 * t));
          mbar_arrive(BAR(B_PFULL + 2 * t + 1));
        } else {
          exp_chunk(r0, 0);
          exp_chunk(r1, 1);
          float s0, s1, s2, s3;
          unpack2(sa, s0, s1);
          unpack2(sb, s2, s3);
          l_run += (s0 + s1) + (s2 + s3);
        }
      }
      const bool in_seq = t_row < s.Nq;  // rows beyond the sequence join the warp-wide loads, only their stores are dropped
      __nv_bfloat16* orow = out + (long long)h * s.os_h + (long long)t_row * s.os_t + ch * OH;
      if (nt == 0) {
        mbar_arrive(BAR(B_OFREE + t));  // keeps the barrier's phase in step with the item count
        for (int c = 0; c < OH / 8 && in_seq; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
        continue;
      }
      // combine the two halves' row sums through the max cells (no longer needed for this item)
      named_bar_sync(pair_bar, 64);
      if (ch == 1) *reinterpret_cast<volatile float*>(mycell) = l_run;
      named_bar_sync(pair_bar, 64);
      const float other1 = *reinterpret_cast<volatile float*>(mycell);
      named_bar_sync(pair_bar, 64);
      if (ch == 0) *reinterpret_cast<volatile float*>(mycell) = l_run;
      named_bar_sync(pair_bar, 64);
      const float other0 = *reinterpret_cast<volatile float*>(mycell);
      l_run += ch ? other0 : other1;
      named_bar_sync(pair_bar, 64);  // both have read the cells: the next item may reset them
      ok = mbar_wait(BAR(B_ODONE + t), (itc - 1) & 1, status);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
#pragma unroll
      for (int c = 0; c < OH / 32; ++c) {
        uint32_t o[32];
        tmem_ld32(t_o + c * 32, o);
        tmem_wait_ld();
        if (c == OH / 32 - 1) {  // O has left tensor memory: the next item's first P.V may overwrite it
          tc_fence_before();
          mbar_arrive(BAR(B_OFREE + t));
        }
#pragma unroll
        for (int v4 = 0; v4 < 4; ++v4) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(o[v4 * 8 + 2 * e]) * inv,
                                                     __uint_as_float(o[v4 * 8 + 2 * e + 1]) * inv);
            w[e] = *reinterpret_cast<uint32_t*>(&b);
          }
          if (in_seq && ok) reinterpret_cast<uint4*>(orow)[c * 4 + v4] = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 16) {
    tc_fence_after();
    tmem_dealloc(tmem, TM_COLS);
    // the last CTA to finish puts the item counter back to zero for the next launch
    if (lane == 0) {
      __threadfence();
      if (atomicAdd(sched + 1, 1) == (int)gridDim.x - 1) {
        sched[0] = 0;
        sched[1] = 0;
        __threadfence();
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Host side: tensor maps and launch
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

// bf16 tensor [heads, N, d] (d contiguous) viewed as a 3-D map, box = 64 x rows x 1, 128-byte swizzle
bool make_tensor_map(CUtensorMap* tm, const void* ptr, int d, int N, int heads, int64_t tok_stride,
                     int64_t head_stride, int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[3] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)heads};
  cuuint64_t gstr[2] = {(cuuint64_t)tok_stride * 2, (cuuint64_t)head_stride * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), gdim, gstr, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// (pk != nullptr: one launch over the sequences of a packed batch -- the tensor maps then span the n_tokens rows of
//  the packed tensors, `grid` counts the CTAs of all sequences and s is any one of them, for the strides)
template <int D, int BN, int NS, bool P_SMEM>
static int launch_t(const Shape& s, const AttnArgs& a, cudaStream_t st, const PackedSeq* pk = nullptr, int npk = 0,
                    long long n_tokens = 0, long long packed_grid = 0) {
  using L = AttSmem<D, BN, NS, P_SMEM>;
  static_assert(L::DYN_BYTES <= 232448, "shared memory budget exceeded");
  CUtensorMap tmq, tmk, tmv;
  if (!make_tensor_map(&tmq, a.q, D, pk ? (int)n_tokens : s.Nq, s.H, s.qs_t, s.qs_h, BM) ||
      !make_tensor_map(&tmk, a.k, D, pk ? (int)n_tokens : s.N, s.Hkv, s.ks_t, s.ks_h, BN) ||
      !make_tensor_map(&tmv, a.v, D, pk ? (int)n_tokens : s.N, s.Hkv, s.vs_t, s.vs_h, BN))
    return EI_ERR_CUDA;
  auto kern = sparse_attention_kernel<D, BN, NS, P_SMEM>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES) != cudaSuccess)
    return EI_ERR_CUDA;
  const long long grid = pk ? packed_grid : (long long)s.H * s.C_S * (s.L_S / BM);
  const float scale_log2 = a.scale * 1.4426950408889634f;
  kern<<<(unsigned)grid, ATT_THREADS, L::DYN_BYTES, st>>>(tmq, tmk, tmv, a.out, a.offsets, a.indices, a.status, s,
                                                         scale_log2, pk, npk);
  return cudaGetLastError() == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

template <int D, int BN, int NSLOT>
static int launch_pair_t(const Shape& s, const AttnArgs& a, cudaStream_t st, const PackedSeq* pk = nullptr, int npk = 0,
                         long long n_tokens = 0, long long packed_grid = 0) {
  using L = Att2Smem<D, BN, NSLOT>;
  static_assert(L::DYN_BYTES <= 232448, "shared memory budget exceeded");
  CUtensorMap tmq, tmk, tmv;
  if (!make_tensor_map(&tmq, a.q, D, pk ? (int)n_tokens : s.Nq, s.H, s.qs_t, s.qs_h, BM) ||
      !make_tensor_map(&tmk, a.k, D, pk ? (int)n_tokens : s.N, s.Hkv, s.ks_t, s.ks_h, BN) ||
      !make_tensor_map(&tmv, a.v, D, pk ? (int)n_tokens : s.N, s.Hkv, s.vs_t, s.vs_h, BN))
    return EI_ERR_CUDA;
  auto kern = sparse_attention_pair_kernel<D, BN, NSLOT>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES) != cudaSuccess)
    return EI_ERR_CUDA;
  const long long grid = pk ? packed_grid : (long long)s.H * s.C_S * (s.L_S / (2 * BM));
  const float scale_log2 = a.scale * 1.4426950408889634f;
  kern<<<(unsigned)grid, ATT2_THREADS, L::DYN_BYTES, st>>>(tmq, tmk, tmv, a.out, a.offsets, a.indices, a.status, s,
                                                          scale_log2, pk, npk);
  return cudaGetLastError() == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

template <int D, int BN, int NSLOT>
static int launch_split_t(const Shape& s, const AttnArgs& a, cudaStream_t st) {
  using L = Att3Smem<D, BN, NSLOT>;
  static_assert(L::DYN_BYTES <= 232448, "shared memory budget exceeded");
  CUtensorMap tmq, tmk, tmv;
  if (!make_tensor_map(&tmq, a.q, D, s.Nq, s.H, s.qs_t, s.qs_h, BM) ||
      !make_tensor_map(&tmk, a.k, D, s.N, s.Hkv, s.ks_t, s.ks_h, BN) ||
      !make_tensor_map(&tmv, a.v, D, s.N, s.Hkv, s.vs_t, s.vs_h, BN))
    return EI_ERR_CUDA;
  auto kern = sparse_attention_split_kernel<D, BN, NSLOT>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES) != cudaSuccess)
    return EI_ERR_CUDA;
  const long long grid = (long long)s.H * s.C_S * (s.L_S / (2 * BM));
  const float scale_log2 = a.scale * 1.4426950408889634f;
  kern<<<(unsigned)grid, ATT3_THREADS, L::DYN_BYTES, st>>>(tmq, tmk, tmv, a.out, a.offsets, a.indices, a.status, s,
                                                          scale_log2, a.skip_log2, a.pv_skipped);
  return cudaGetLastError() == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

template <int D, int BN, int NSLOT>
static int launch_persistent_t(const Shape& s, const AttnArgs& a, cudaStream_t st) {
  using L = Att4Smem<D, BN, NSLOT>;
  static_assert(L::DYN_BYTES <= 232448, "shared memory budget exceeded");
  CUtensorMap tmq, tmk, tmv;
  if (!make_tensor_map(&tmq, a.q, D, s.Nq, s.H, s.qs_t, s.qs_h, BM) ||
      !make_tensor_map(&tmk, a.k, D, s.N, s.Hkv, s.ks_t, s.ks_h, BN) ||
      !make_tensor_map(&tmv, a.v, D, s.N, s.Hkv, s.vs_t, s.vs_h, BN))
    return EI_ERR_CUDA;
  auto kern = sparse_attention_persistent_kernel<D, BN, NSLOT>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES) != cudaSuccess)
    return EI_ERR_CUDA;
  const long long n_items = (long long)s.H * s.C_S * (s.L_S / (2 * BM));
  const unsigned grid = (unsigned)(n_items < 148 ? n_items : 148);  // one CTA per SM; items come off a counter
  const float scale_log2 = a.scale * 1.4426950408889634f;
  kern<<<grid, ATT3_THREADS, L::DYN_BYTES, st>>>(tmq, tmk, tmv, a.out, a.offsets, a.indices, a.status, a.sched, s,
                                               scale_log2, a.skip_log2, (int)n_items);
  return cudaGetLastError() == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

// The sequences of a packed batch in one launch, by the kernel launch_attention would pick for each of them without
// flags: the quad-layout kernel (d = 128, 128-wide blocks, segments a multiple of 256), else a two-tile kernel
// (segments a multiple of 256), else the one-tile kernel.  pk_host[i].w_att (packed_fill_work) counts the CTAs of the
// earlier sequences accordingly.
int launch_attention_packed(const PackedSeq* pk, const PackedSeq* pk_host, int npk, long long n_tokens, const AttnArgs& a,
                            cudaStream_t st) {
  const Shape& s = pk_host[npk - 1].s;
  const bool pairs = s.L_S % (2 * BM) == 0 && s.d != 256;
  const long long grid = pk_host[npk - 1].w_att + (long long)s.H * s.C_S * (s.L_S / (pairs ? 2 * BM : BM));
  if (pairs && s.d == 128 && s.L_B == 128) return launch_attention_quad_packed(pk, pk_host, npk, n_tokens, a, st);
  if (s.d == 256) {
    if (s.L_B == 128) return launch_t<256, 128, 1, false>(s, a, st, pk, npk, n_tokens, grid);
    return launch_t<256, 64, 2, false>(s, a, st, pk, npk, n_tokens, grid);
  }
  if (pairs) {
    if (s.d == 128 && s.L_B == 64) return launch_pair_t<128, 64, 6>(s, a, st, pk, npk, n_tokens, grid);
    if (s.d == 64 && s.L_B == 128) return launch_pair_t<64, 128, 6>(s, a, st, pk, npk, n_tokens, grid);
    if (s.d == 64 && s.L_B == 64) return launch_pair_t<64, 64, 6>(s, a, st, pk, npk, n_tokens, grid);
  }
  if (s.d == 128 && s.L_B == 128) return launch_t<128, 128, 3, false>(s, a, st, pk, npk, n_tokens, grid);
  if (s.d == 128 && s.L_B == 64) return launch_t<128, 64, 4, false>(s, a, st, pk, npk, n_tokens, grid);
  if (s.d == 64 && s.L_B == 128) return launch_t<64, 128, 4, false>(s, a, st, pk, npk, n_tokens, grid);
  if (s.d == 64 && s.L_B == 64) return launch_t<64, 64, 4, false>(s, a, st, pk, npk, n_tokens, grid);
  return EI_ERR_UNSUPPORTED_SHAPE;
}

int launch_attention(const Shape& s, const AttnArgs& a, cudaStream_t st) {
  // head_dim 256: S (128 columns, twice) and O (256 columns) fill the tensor memory of an SM, so a CTA owns one
  // 128-row tile; Q, one K and one V tile (64 KB each at 128-wide blocks) fill its shared memory
  if (s.d == 256) {
    if (s.L_B == 128) return launch_t<256, 128, 1, false>(s, a, st);
    if (s.L_B == 64) return launch_t<256, 64, 2, false>(s, a, st);
    return EI_ERR_UNSUPPORTED_SHAPE;
  }
  if (a.tri_kernel && s.L_S % (2 * BM) == 0 && s.d == 128 && s.L_B == 128) return launch_attention_tri(s, a, st);
  if (a.quad_kernel && s.L_S % (2 * BM) == 0 && s.d == 128 && s.L_B == 128) return launch_attention_quad(s, a, st);
  if (a.persistent && a.sched && s.L_S % (2 * BM) == 0 && s.d == 128 && s.L_B == 128)
    return launch_persistent_t<128, 128, 5>(s, a, st);

  // d = 128, 128-wide key blocks, segments of a multiple of 256 rows: the split-row kernel
  if (!a.p_via_smem && !a.single_tile && !a.pair_8warp && s.L_S % (2 * BM) == 0 && s.d == 128 && s.L_B == 128)
    return launch_split_t<128, 128, 5>(s, a, st);
  if (!a.p_via_smem && !a.single_tile && s.L_S % (2 * BM) == 0) {
    if (s.d == 128 && s.L_B == 128) return launch_pair_t<128, 128, 5>(s, a, st);
    if (s.d == 128 && s.L_B == 64) return launch_pair_t<128, 64, 6>(s, a, st);
    if (s.d == 64 && s.L_B == 128) return launch_pair_t<64, 128, 6>(s, a, st);
    if (s.d == 64 && s.L_B == 64) return launch_pair_t<64, 64, 6>(s, a, st);
  }
  if (s.d == 128 && s.L_B == 128) return a.p_via_smem ? launch_t<128, 128, 2, true>(s, a, st) : launch_t<128, 128, 3, false>(s, a, st);
  if (s.d == 128 && s.L_B == 64) return a.p_via_smem ? launch_t<128, 64, 4, true>(s, a, st) : launch_t<128, 64, 4, false>(s, a, st);
  if (s.d == 64 && s.L_B == 128) return a.p_via_smem ? launch_t<64, 128, 4, true>(s, a, st) : launch_t<64, 128, 4, false>(s, a, st);
  if (s.d == 64 && s.L_B == 64) return a.p_via_smem ? launch_t<64, 64, 4, true>(s, a, st) : launch_t<64, 64, 4, false>(s, a, st);
  return EI_ERR_UNSUPPORTED_SHAPE;
}

}  // namespace ei
