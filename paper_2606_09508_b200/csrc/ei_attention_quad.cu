// Stage 4, quad-layout kernels: causal GQA flash attention over the selected key blocks (Eq. t_spa) for
// head_dim 128 and 128-wide key blocks, hand-written for sm_100a.
//
// A CTA works on two adjacent 128-row query tiles of a (head, segment) cell at a time.  Sixteen softmax warps
// share the work so that no key block needs an exchange between warps: a warp owns SIXTEEN query rows
// (tensor-memory lanes) and all 128 key columns, read with the 16-lane tensor-memory shape
// (tcgen05.ld.16x256b), in which the four threads of a quad hold one row pair: thread t has rows t/4 and
// t/4 + 8, columns 8i + 2(t%4), +1 of every 8-column group i.  The row maximum is a max over the thread's 32
// values and two shuffles inside the quad; the probabilities go back as bf16 pairs with the matching store
// shape (tcgen05.st.16x128b).  The two warps of a 32-lane quadrant run independently of each other.
//
//   warps 0-7   tile 0: warp w -> lanes 32*(w%4) + 16*(w/4) .. +15
//   warps 8-15  tile 1
//   warp 16     TMA producer          warp 17   MMA issuer          warp 18   scheduler (persistent form only)
//
// Tensor memory: S0 at 0, S1 at 128, O0 at 256, O1 at 384 (fp32); P (bf16 pairs) overwrites the first 64
// columns of its tile's S and is handed to the MMA warp in two halves (keys 0-63, then 64-127), so P.V starts
// while the second half is still being exponentiated.
//
// Two forms.  sparse_attention_quad_kernel: one CTA per tile pair.  sparse_attention_quad_persistent_kernel:
// one CTA per SM for the whole launch; a scheduler warp takes (head, segment, tile pair) items off a global
// counter (long block lists first), looks the block list up and publishes a small record per item in a ring of
// four, so that the producer can load the next item's Q and first K/V tiles, the MMA warp can issue its first
// Q.K^T and the softmax warps can start on it while the previous item's output is still being written.
// Every mbarrier wait is bounded; on expiry the status word is set, later waits return at once, and the CTA
// drains its loads and frees its tensor memory.
#include <cuda.h>

#include "ei_internal.cuh"
#include "ei_sm100.cuh"

namespace ei {

constexpr int QUAD_THREADS = 576;
constexpr int QUADP_THREADS = 608;
constexpr int QBM = 128;
constexpr float QUAD_RESCALE_THRESHOLD = 8.0f;  // log2 units
__host__ __device__ constexpr uint32_t qtm_s(int t) { return 128u * (uint32_t)t; }
__host__ __device__ constexpr uint32_t qtm_o(int t) { return 256u + 128u * (uint32_t)t; }
constexpr uint32_t QTM_COLS = 512;

// 16 lanes x 64 columns of fp32: r[4i + {0,1}] = row t/4, columns 8i + 2(t%4) + {0,1}; r[4i + {2,3}] = row t/4 + 8
__device__ __forceinline__ void tmem_ld_16x64(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// 16 lanes x 32 packed columns (64 bf16): r[2i] = row t/4, packed column 4i + t%4; r[2i + 1] = row t/4 + 8
__device__ __forceinline__ void tmem_st_16x32(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.16x128b.x8.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
      ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_16x8(uint32_t taddr, uint32_t (&r)[4]) {
  asm volatile("tcgen05.ld.sync.aligned.16x256b.x1.b32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_st_16x8(uint32_t taddr, const uint32_t (&r)[4]) {
  asm volatile("tcgen05.st.sync.aligned.16x256b.x1.b32 [%4], {%0,%1,%2,%3};" ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]),
               "r"(taddr)
               : "memory");
}

// running state of a thread's two query rows: reference maxima (raw logit units) and partial row sums
struct QuadRows {
  float mrA, mrB, lA, lB;
};

// O[my two rows, all columns] *= alpha, once the P.V products issued so far have landed (rare: only when a row's
// maximum moved by more than 2^8).  Out of line: its registers and loop stay out of the softmax loop.
template <int D>
__device__ __noinline__ bool quad_rescale(uint32_t t_o, float alA, float alB, uint32_t bar_odone, uint32_t par, int* status) {
  bool ok = mbar_wait(bar_odone, par, status);
  ok = __all_sync(0xffffffffu, ok);
  tc_fence_after();
#pragma unroll 1
  for (int c = 0; c < D / 8; ++c) {  // eight columns at a time
    uint32_t o[4];
    tmem_ld_16x8(t_o + c * 8, o);
    tmem_wait_ld();
    o[0] = __float_as_uint(__uint_as_float(o[0]) * alA);
    o[1] = __float_as_uint(__uint_as_float(o[1]) * alA);
    o[2] = __float_as_uint(__uint_as_float(o[2]) * alB);
    o[3] = __float_as_uint(__uint_as_float(o[3]) * alB);
    tmem_st_16x8(t_o + c * 8, o);
  }
  return ok;
}

// One key block of the online softmax for the 16 rows of a warp.  Waits for S, reads it, updates the reference
// maxima (rescaling O when a row's maximum moved by more than 2^8), writes P and hands its two halves over.
//   first:   the tile's first block of the item (the references are taken from it, O holds nothing yet)
//   limA:    causal bound for row A in units of my column offsets (INT_MAX when the block needs no mask): key
//            column c of the block is visible to row A iff c - 2*(lane%4) <= limA, to row B iff <= limA + 8
template <int D, int BN, bool SKIP>
__device__ __forceinline__ bool quad_softmax_block(uint32_t t_s, uint32_t t_o, uint32_t bar_sfull, uint32_t par_sfull,
                                                   uint32_t bar_odone, uint32_t par_odone_prev, uint32_t bar_p0,
                                                   uint32_t bar_p1, bool first, bool masked, int limA,
                                                   float scale_log2, float skip_log2, int lane, int* status,
                                                   QuadRows& st) {
  bool ok = mbar_wait(bar_sfull, par_sfull, status);
  ok = __all_sync(0xffffffffu, ok);
  tc_fence_after();
  uint32_t xa[32], xb[32];  // columns 0..63 and 64..127: [4i + {0,1}] row A, [4i + {2,3}] row B, columns 8i + 2*(lane%4) + {0,1}
  tmem_ld_16x64(t_s, xa);
  tmem_ld_16x64(t_s + 64, xb);
  tmem_wait_ld();
  if (masked) {
#pragma unroll
    for (int ii = 0; ii < 8; ++ii) {
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        if (8 * ii + k > limA) xa[4 * ii + k] = 0xff800000u;
        if (8 * ii + k > limA + 8) xa[4 * ii + 2 + k] = 0xff800000u;
        if (64 + 8 * ii + k > limA) xb[4 * ii + k] = 0xff800000u;
        if (64 + 8 * ii + k > limA + 8) xb[4 * ii + 2 + k] = 0xff800000u;
      }
    }
  }
  // maxima of my 32 values per row (two chains per row), then over the quad
  float mA0 = __uint_as_float(xa[0]), mA1 = __uint_as_float(xa[1]), mB0 = __uint_as_float(xa[2]),
        mB1 = __uint_as_float(xa[3]);
#pragma unroll
  for (int ii = 1; ii < 8; ii += 2) {
    mA0 = fmax3(mA0, __uint_as_float(xa[4 * ii]), __uint_as_float(xa[4 * ii + 1]));
    mB0 = fmax3(mB0, __uint_as_float(xa[4 * ii + 2]), __uint_as_float(xa[4 * ii + 3]));
    if (ii + 1 < 8) {
      mA1 = fmax3(mA1, __uint_as_float(xa[4 * ii + 4]), __uint_as_float(xa[4 * ii + 5]));
      mB1 = fmax3(mB1, __uint_as_float(xa[4 * ii + 6]), __uint_as_float(xa[4 * ii + 7]));
    }
  }
#pragma unroll
  for (int ii = 0; ii < 8; ii += 2) {
    mA1 = fmax3(mA1, __uint_as_float(xb[4 * ii]), __uint_as_float(xb[4 * ii + 1]));
    mB1 = fmax3(mB1, __uint_as_float(xb[4 * ii + 2]), __uint_as_float(xb[4 * ii + 3]));
    mA0 = fmax3(mA0, __uint_as_float(xb[4 * ii + 4]), __uint_as_float(xb[4 * ii + 5]));
    mB0 = fmax3(mB0, __uint_as_float(xb[4 * ii + 6]), __uint_as_float(xb[4 * ii + 7]));
  }
  float lmA = fmaxf(mA0, mA1), lmB = fmaxf(mB0, mB1);
  lmA = fmaxf(lmA, __shfl_xor_sync(0xffffffffu, lmA, 1));
  lmB = fmaxf(lmB, __shfl_xor_sync(0xffffffffu, lmB, 1));
  lmA = fmaxf(lmA, __shfl_xor_sync(0xffffffffu, lmA, 2));  // the largest logit of row A in this block
  lmB = fmaxf(lmB, __shfl_xor_sync(0xffffffffu, lmB, 2));
  if (first) {
    st.mrA = lmA;
    st.mrB = lmB;
  } else {
    const bool needA = (lmA - st.mrA) * scale_log2 > QUAD_RESCALE_THRESHOLD;  // a reference of -inf: inf > 8
    const bool needB = (lmB - st.mrB) * scale_log2 > QUAD_RESCALE_THRESHOLD;
    if (__any_sync(0xffffffffu, needA || needB)) {
      const float alA = needA ? fast_ex2((st.mrA - lmA) * scale_log2) : 1.0f;
      const float alB = needB ? fast_ex2((st.mrB - lmB) * scale_log2) : 1.0f;
      ok = quad_rescale<D>(t_o, alA, alB, bar_odone, par_odone_prev, status) && ok;
      st.lA *= alA;
      st.lB *= alB;
      if (needA) st.mrA = lmA;
      if (needB) st.mrB = lmB;
    }
  }
  // Rows whose largest logit lies more than skip_log2 binary orders below the reference maximum hold only terms
  // below 2^-skip_log2 of the row's largest: where that is so for all 16 rows of the warp, P is zero and nothing
  // is exponentiated.  (A fully masked row, -inf, qualifies; a reference of -inf gives NaN: not.)
  if (SKIP && __all_sync(0xffffffffu,
                         (lmA - st.mrA) * scale_log2 < -skip_log2 && (lmB - st.mrB) * scale_log2 < -skip_log2)) {
    uint32_t(&zero)[16] = *reinterpret_cast<uint32_t(*)[16]>(&xa[0]);
#pragma unroll
    for (int e = 0; e < 16; ++e) zero[e] = 0u;
    tmem_st_16x32(t_s, zero);
    tmem_st_16x32(t_s + 32, zero);
    tmem_wait_st();
    tc_fence_before();
    __syncwarp();
    if (lane == 0) {
      mbar_arrive(bar_p0);
      mbar_arrive(bar_p1);
    }
    return ok;
  }
  // P = exp2(s * scale - m * scale), partial row sums, bf16 pairs over the first 64 columns of S.  The packed
  // pair e of a half goes back into register e of that half's own array (its inputs 2e, 2e+1 are read before),
  // so the sixteen registers handed to the store are the array's first sixteen and P needs no registers of its own.
  const float mcA = (st.mrA == -INFINITY) ? 0.f : st.mrA * scale_log2;
  const float mcB = (st.mrB == -INFINITY) ? 0.f : st.mrB * scale_log2;
  const uint64_t c2 = pack2(scale_log2, scale_log2), nmA = pack2(-mcA, -mcA), nmB = pack2(-mcB, -mcB);
  uint64_t sA = 0ull, sB = 0ull;
#pragma unroll
  for (int part = 0; part < 2; ++part) {
    uint32_t(&x)[32] = part ? xb : xa;
#pragma unroll
    for (int e = 0; e < 16; ++e) {  // pair e: row A when even, row B when odd
      float a0, a1;
      unpack2(ffma2(pack2(__uint_as_float(x[2 * e]), __uint_as_float(x[2 * e + 1])), c2, (e & 1) ? nmB : nmA), a0, a1);
      a0 = fast_ex2(a0);
      a1 = fast_ex2(a1);
      if (e & 1) sB = fadd2(sB, pack2(a0, a1));
      else sA = fadd2(sA, pack2(a0, a1));
      __nv_bfloat162 pb = __floats2bfloat162_rn(a0, a1);
      x[e] = *reinterpret_cast<uint32_t*>(&pb);
    }
    tmem_st_16x32(t_s + part * 32, *reinterpret_cast<uint32_t(*)[16]>(&x[0]));
    tmem_wait_st();
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(part ? bar_p1 : bar_p0);
  }
  float s0, s1;
  unpack2(sA, s0, s1);
  st.lA += s0 + s1;
  unpack2(sB, s0, s1);
  st.lB += s0 + s1;
  return ok;
}

// Row sums across the quad, published per row; then the warp's share of the output: 32 rows x 64 columns of
// O / l as bf16 (32-lane shape: thread = row; the two warps of a quadrant take one half of the columns each).
// lsum: float [128] of this tile; pair_bar: named barrier of the quadrant's two warps; returns after the O loads
// have completed (o_read is then signalled by the caller) -- the stores follow.
template <int D>
__device__ __forceinline__ void quad_epilogue_sums(QuadRows& st, float* lsum, int rowA, int q4, int pair_bar) {
  st.lA += __shfl_xor_sync(0xffffffffu, st.lA, 1);
  st.lB += __shfl_xor_sync(0xffffffffu, st.lB, 1);
  st.lA += __shfl_xor_sync(0xffffffffu, st.lA, 2);
  st.lB += __shfl_xor_sync(0xffffffffu, st.lB, 2);
  if (q4 == 0) {
    lsum[rowA] = st.lA;
    lsum[rowA + 8] = st.lB;
  }
  asm volatile("bar.sync %0, %1;" ::"r"(pair_bar), "r"(64) : "memory");  // the two warps of this quadrant
}

// My row's share of the output: COLS columns of O / l as bf16 (32-lane shape: thread = row).  Signals o_read
// once the last tensor-memory load has completed.  Out of line: it runs once per item and its staging registers
// must not weigh on the softmax loop of the persistent kernel.
template <int COLS>
__device__ __noinline__ void quad_store_rows(uint32_t t_o32, __nv_bfloat16* orow, float inv, bool store, uint32_t bar_oread,
                                             int lane) {
#pragma unroll
  for (int c = 0; c < COLS / 32; ++c) {
    uint32_t o[32];
    tmem_ld32(t_o32 + c * 32, o);
    tmem_wait_ld();
    if (c == COLS / 32 - 1) {  // O has left tensor memory: the next item's first P.V may overwrite it
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_oread);
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
      if (store) reinterpret_cast<uint4*>(orow)[c * 4 + v4] = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

template <int D, int BN, int NSLOT>
struct QuadSmem {
  static constexpr int Q_BYTES = QBM * D * 2;
  static constexpr int KV_BYTES = BN * D * 2;
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_RING = 2 * Q_BYTES;
  static constexpr int OFF_LSUM = OFF_RING + NSLOT * KV_BYTES;  // float [2 tiles][128 rows]: row sums for the epilogue
  static constexpr int OFF_REC = OFF_LSUM + 2 * QBM * 4;        // int [4 records][8] (persistent form)
  static constexpr int OFF_BAR = OFF_REC + 4 * 8 * 4;
  // q_full[2] q_empty[2] ring full/empty s_full[2] p_full[4] o_done[2] o_read[2] rec_full[4] rec_empty[4]
  static constexpr int NBAR = 4 + 2 * NSLOT + 2 + 4 + 2 + 2 + 8;
  static constexpr int TOTAL = OFF_BAR + NBAR * 8 + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;
};

// ------------------------------------------------------------------------------------------------
// One CTA per tile pair
// ------------------------------------------------------------------------------------------------
template <int D, int BN, int NSLOT, bool SKIP>
__global__ void __maxnreg__(96)
sparse_attention_quad_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                             const __grid_constant__ CUtensorMap tmv, __nv_bfloat16* __restrict__ out,
                             const int* __restrict__ items, const int* __restrict__ indices,
                             int* __restrict__ status, Shape s, float scale_log2, float skip_log2,
                             const PackedSeq* pk, int npk) {
  using L = QuadSmem<D, BN, NSLOT>;
  static_assert(BN == 128 && D == 128, "the quad-layout kernels are written for head_dim 128 and 128-wide key blocks");
  extern __shared__ unsigned char att_smem_raw[];

  const uint32_t raw = smem_u32(att_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gbase = att_smem_raw + (base - raw);
  const uint32_t sQ = base + L::OFF_Q, sRing = base + L::OFF_RING;
  float* lsum = reinterpret_cast<float*>(gbase + L::OFF_LSUM);
  const uint32_t bar0 = base + L::OFF_BAR;
  auto BAR = [&](int i) { return bar0 + 8u * i; };
  const int B_QFULL = 0, B_FULL = 4, B_EMPTY = 4 + NSLOT, B_SFULL = 4 + 2 * NSLOT, B_PFULL = B_SFULL + 2,
            B_ODONE = B_PFULL + 4;  // p_full: index 2*t + part
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gbase + L::OFF_BAR + L::NBAR * 8);

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);

  const int pairs_per_seg = s.L_S / (2 * QBM);
  int bid = blockIdx.x;
  int tok0 = 0;  // a packed batch: my sequence starts here in q, k, v, out (the tensor maps span the whole batch)
  if (pk != nullptr) {
    const PackedSeq& P = pk[packed_find(pk, npk, bid, &PackedSeq::w_att)];
    s = P.s;
    bid -= P.w_att;
    tok0 = (int)P.tok0;
    items += P.lcell0 * pairs_per_seg * 8;
    indices += P.idx0;
    out += P.tok0 * s.os_t;
  }
  const int pr = bid % pairs_per_seg;
  bid /= pairs_per_seg;
  const int h = bid % s.H;
  const int i = s.C_S - 1 - bid / s.H;  // long lists (late segments) first
  const int g = h / s.G;
  const long long cell = (long long)(h / s.list_div) * s.C_S + i;
  const int q0 = i * s.L_S + pr * 2 * QBM;
  if (q0 >= s.Nq) return;  // a pair of tiles of the short last segment that lies beyond the sequence (CTA-uniform)

  // The producer warp initialises the barriers and starts the Q loads (they depend only on the block index)
  // before anyone has read the block list, so the first tiles are in flight during set-up.
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
        mbar_init(BAR(B_PFULL + 2 * t), 8);  // one arrival per softmax warp of the tile
        mbar_init(BAR(B_PFULL + 2 * t + 1), 8);
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
        tma_load_3d(sQ + t * L::Q_BYTES + p * (QBM * 128), &tmq, p * 64, tok0 + q0 + t * QBM, h, BAR(B_QFULL + t));
    }
  }
  // my item's record: list offset, blocks visible to tile 0 / tile 1, first masked entry of either, first block
  const int4* recp = reinterpret_cast<const int4*>(items + (cell * pairs_per_seg + pr) * 8);
  const int4 r0 = __ldg(recp), r1 = __ldg(recp + 1);
  const int off = r0.x, n0 = r0.y, n1 = r0.z, blk0 = r1.y;

  // ring items: K_j is item 2j, V_j is item 2j+1; the first NSLOT need no free-slot wait
  auto load_item = [&](int u, int blk) {
    const int slot = u % NSLOT;
    mbar_expect_tx(BAR(B_FULL + slot), L::KV_BYTES);
    const CUtensorMap* tm = (u & 1) ? &tmv : &tmk;
#pragma unroll
    for (int p = 0; p < D / 64; ++p)
      tma_load_3d(sRing + slot * L::KV_BYTES + p * (BN * 128), tm, p * 64, tok0 + blk * BN, g, BAR(B_FULL + slot));
  };
  int issued = 0;
  // testing aid (ei_plan_debug_waits): one ring item the producer leaves out, so that a bounded wait runs out
  const int skip_item = warp == 16 ? reinterpret_cast<volatile int*>(status)[2] - 1 : -1;
  if (warp == 16 && n1 > 0) {
    for (int u = 0; u < 2 * n1 && u < NSLOT; ++u) {
      if (u != skip_item) load_item(u, u < 2 ? blk0 : __ldg(indices + off + (u >> 1)));
      issued = u + 1;
    }
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), QTM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // (a cell without any visible key -- only possible with hand-made lists -- runs through the same roles with
  //  n1 = 0: the producer only lets its Q loads land, the MMA warp issues nothing, the softmax threads write zeros)
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
    if (n1 > 0) {
      // ================= MMA issuer (whole warp, elected lane issues) =================
      constexpr uint32_t IDESC_QK = make_idesc(BN, false);
      constexpr uint32_t IDESC_PV = make_idesc(D, true);
      auto wait_item = [&](int u) { return mbar_wait(BAR(B_FULL + u % NSLOT), (u / NSLOT) & 1, status); };
      auto issue_qk = [&](int t, int j) {  // S_t = Q_t . K_j^T
        const uint32_t kbase = sRing + ((2 * j) % NSLOT) * L::KV_BYTES;
        const uint32_t qbase = sQ + t * L::Q_BYTES;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint64_t ad = make_desc(qbase + (ks / 4) * (QBM * 128) + (ks % 4) * 32, 16, 1024);
          const uint64_t bd = make_desc(kbase + (ks / 4) * (BN * 128) + (ks % 4) * 32, 16, 1024);
          umma_ss(tmem + qtm_s(t), ad, bd, IDESC_QK, ks > 0 ? 1u : 0u);
        }
        umma_commit(BAR(B_SFULL + t));
      };
      // O_t += P_t . V_j in two halves: part 0 = keys 0..63 of the block, part 1 = keys 64..127
      auto issue_pv = [&](int t, int j, int part) {
        const uint32_t vbase = sRing + ((2 * j + 1) % NSLOT) * L::KV_BYTES;
        constexpr int HALF = BN / 32;
#pragma unroll
        for (int u = 0; u < HALF; ++u) {
          const int ks = part * HALF + u;
          const uint64_t bd = make_desc(vbase + ks * 2048, BN * 128, 1024);
          umma_ts(tmem + qtm_o(t), tmem + qtm_s(t) + ks * 8, bd, IDESC_PV, (j > 0 || part > 0 || u > 0) ? 1u : 0u);
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
        for (int j = 0; j < n1 && ok; ++j) {
          if (j < n0) {
            if (!(ok = mbar_wait(BAR(B_PFULL), j & 1, status))) break;
            if (!(ok = wait_item(2 * j + 1))) break;
            tc_fence_after();
            issue_pv(0, j, 0);
            if (!(ok = mbar_wait(BAR(B_PFULL + 1), j & 1, status))) break;
            tc_fence_after();
            issue_pv(0, j, 1);
            if (j + 1 < n0) {
              if (!(ok = wait_item(2 * j + 2))) break;
              tc_fence_after();
              issue_qk(0, j + 1);
            }
          }
          if (!(ok = mbar_wait(BAR(B_PFULL + 2), j & 1, status))) break;
          if (!(ok = wait_item(2 * j + 1))) break;
          tc_fence_after();
          issue_pv(1, j, 0);
          if (!(ok = mbar_wait(BAR(B_PFULL + 3), j & 1, status))) break;
          tc_fence_after();
          issue_pv(1, j, 1);
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
    // ================= softmax: tile t = warp / 8, 16 rows per warp, a row pair per quad of threads =================
    // (after a timed-out wait the threads keep going through the motions: later waits return at once)
    const int t = warp >> 3;
    const int nt = t ? n1 : n0;
    const int qd = warp & 3, hf = (warp >> 2) & 1;
    const int q4 = lane & 3;
    const int rowA = qd * 32 + hf * 16 + (lane >> 2);  // my two rows of the tile: rowA and rowA + 8
    const uint32_t lane16 = (uint32_t)(qd * 32 + hf * 16) << 16;
    const int tq0 = q0 + t * QBM;
    const uint32_t t_s = tmem + lane16 + qtm_s(t);
    const uint32_t t_o = tmem + lane16 + qtm_o(t);
    const int jm = t ? r1.x : r0.w;  // only blocks reaching past the tile's first row need the causal mask: entries j >= jm
    QuadRows st = {-INFINITY, -INFINITY, 0.f, 0.f};
    for (int j = 0; j < nt; ++j) {
      const bool masked = j >= jm;
      const int limA = masked ? rowA + tq0 + s.P - __ldg(indices + off + j) * BN - 2 * q4 : 0x7fffffff - 8;
      ok = quad_softmax_block<D, BN, SKIP>(t_s, t_o, BAR(B_SFULL + t), j & 1, BAR(B_ODONE + t), (j - 1) & 1,
                                     BAR(B_PFULL + 2 * t), BAR(B_PFULL + 2 * t + 1), j == 0, masked, limA, scale_log2,
                                     skip_log2, lane, status, st) && ok;
    }
    quad_epilogue_sums<D>(st, lsum + t * QBM, rowA, q4, 1 + t * 4 + qd);
    const int row = qd * 32 + lane;
    const float l_row = lsum[t * QBM + row];
    if (nt > 0) {
      ok = mbar_wait(BAR(B_ODONE + t), (nt - 1) & 1, status) && ok;
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      const int t_row = tq0 + row;
      const bool in_seq = t_row < s.Nq;  // rows beyond the sequence join the warp-wide loads, only their stores are dropped
      constexpr int OH = D / 2;
      __nv_bfloat16* orow = out + (long long)h * s.os_h + (long long)t_row * s.os_t + hf * OH;
      if (nt == 0) {
        for (int c = 0; c < OH / 8 && in_seq; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
      } else {
        tc_fence_after();
        const float inv = l_row > 0.f ? 1.0f / l_row : 0.f;
        const uint32_t t_o32 = tmem + ((uint32_t)(qd * 32) << 16) + qtm_o(t) + hf * OH;
#pragma unroll
        for (int c = 0; c < OH / 32; ++c) {
          uint32_t o[32];
          tmem_ld32(t_o32 + c * 32, o);
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
  if (warp == 16 && n1 > 0) {
    tc_fence_after();
    tmem_dealloc(tmem, QTM_COLS);
  }
}

// ------------------------------------------------------------------------------------------------
// One 128-row tile per CTA, two CTAs per SM.  Each CTA takes half of the tensor memory (S at column 0, O at
// 128) and half of the shared memory (Q + one K slot + one V slot), eight softmax warps, a producer and an MMA
// warp; the hardware interleaves the two CTAs of an SM, so one CTA's set-up, softmax and output phases run
// under the other one's tensor-core work without any hand-written ordering between the tiles.  The price is
// that the two tiles no longer share their K/V tiles in shared memory (each CTA loads its own; the second
// request hits in L2).
// ------------------------------------------------------------------------------------------------
constexpr int QUAD1_THREADS = 320;
constexpr uint32_t QTM1_COLS = 256, QTM1_S = 0, QTM1_O = 128;

template <int D, int BN>
struct Quad1Smem {
  static constexpr int Q_BYTES = QBM * D * 2;
  static constexpr int KV_BYTES = BN * D * 2;
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = Q_BYTES;
  static constexpr int OFF_V = OFF_K + KV_BYTES;
  static constexpr int OFF_LSUM = OFF_V + KV_BYTES;  // float [128 rows]
  static constexpr int OFF_BAR = OFF_LSUM + QBM * 4;
  static constexpr int NBAR = 1 + 4 + 1 + 2 + 1;  // q_full, k_full, v_full, k_empty, v_empty, s_full, p_full[2], o_done
  static constexpr int TOTAL = OFF_BAR + NBAR * 8 + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;
};

template <int D, int BN, bool SKIP>
__global__ void __launch_bounds__(QUAD1_THREADS, 2)
sparse_attention_quad1_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                              const __grid_constant__ CUtensorMap tmv, __nv_bfloat16* __restrict__ out,
                              const int* __restrict__ items, const int* __restrict__ indices,
                              int* __restrict__ status, Shape s, float scale_log2, float skip_log2) {
  using L = Quad1Smem<D, BN>;
  static_assert(BN == 128 && D == 128, "the quad-layout kernels are written for head_dim 128 and 128-wide key blocks");
  extern __shared__ unsigned char att_smem_raw[];

  const uint32_t raw = smem_u32(att_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gbase = att_smem_raw + (base - raw);
  const uint32_t sQ = base + L::OFF_Q, sK = base + L::OFF_K, sV = base + L::OFF_V;
  float* lsum = reinterpret_cast<float*>(gbase + L::OFF_LSUM);
  const uint32_t bar0 = base + L::OFF_BAR;
  auto BAR = [&](int i) { return bar0 + 8u * i; };
  const int B_QFULL = 0, B_KFULL = 1, B_VFULL = 2, B_KEMPTY = 3, B_VEMPTY = 4, B_SFULL = 5, B_PFULL = 6, B_ODONE = 8;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gbase + L::OFF_BAR + L::NBAR * 8);

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);

  const int tiles_per_seg = s.L_S / QBM, pairs_per_seg = tiles_per_seg / 2;
  int bid = blockIdx.x;
  const int tt = bid % tiles_per_seg;
  bid /= tiles_per_seg;
  const int h = bid % s.H;
  const int i = s.C_S - 1 - bid / s.H;  // long lists (late segments) first
  const int g = h / s.G;
  const long long cell = (long long)(h / s.list_div) * s.C_S + i;
  const int tq0 = i * s.L_S + tt * QBM;
  if (tq0 >= s.Nq) return;  // a tile of the short last segment that lies beyond the sequence (CTA-uniform)

  if (warp == 8) {
    if (lane == 0) {
      mbar_init(BAR(B_QFULL), 1);
      mbar_init(BAR(B_KFULL), 1);
      mbar_init(BAR(B_VFULL), 1);
      mbar_init(BAR(B_KEMPTY), 1);
      mbar_init(BAR(B_VEMPTY), 1);
      mbar_init(BAR(B_SFULL), 1);
      mbar_init(BAR(B_PFULL), 8);  // one arrival per softmax warp
      mbar_init(BAR(B_PFULL + 1), 8);
      mbar_init(BAR(B_ODONE), 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      fence_async_smem();
    }
    __syncwarp();
    mbar_expect_tx(BAR(B_QFULL), L::Q_BYTES);
#pragma unroll
    for (int p = 0; p < D / 64; ++p) tma_load_3d(sQ + p * (QBM * 128), &tmq, p * 64, tq0, h, BAR(B_QFULL));
  }
  // my tile's share of the pair's record
  const int4* recp = reinterpret_cast<const int4*>(items + (cell * pairs_per_seg + (tt >> 1)) * 8);
  const int4 r0 = __ldg(recp), r1 = __ldg(recp + 1);
  const int off = r0.x, nt = (tt & 1) ? r0.z : r0.y, jm = (tt & 1) ? r1.x : r0.w, blk0 = r1.y;

  auto load_kv = [&](bool is_v, int blk) {
    const uint32_t bar = BAR(is_v ? B_VFULL : B_KFULL);
    mbar_expect_tx(bar, L::KV_BYTES);
#pragma unroll
    for (int p = 0; p < D / 64; ++p)
      tma_load_3d((is_v ? sV : sK) + p * (BN * 128), is_v ? &tmv : &tmk, p * 64, blk * BN, g, bar);
  };
  if (warp == 8 && nt > 0) {
    load_kv(false, blk0);
    load_kv(true, blk0);
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), QTM1_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  bool ok = true;

  if (warp == 8) {
    // ================= TMA producer: K_j into the K slot once Q.K^T_{j-1} has read it, V_j likewise =================
    int kdone = nt > 0 ? 1 : 0, vdone = kdone;  // loads issued so far
    for (int j = 1; j < nt; ++j) {
      const int blk = __ldg(indices + off + j);
      ok = mbar_wait(BAR(B_KEMPTY), (j - 1) & 1, status);
      if (!ok) break;
      load_kv(false, blk);
      kdone = j + 1;
      ok = mbar_wait(BAR(B_VEMPTY), (j - 1) & 1, status);
      if (!ok) break;
      load_kv(true, blk);
      vdone = j + 1;
    }
    // Drain: every load issued here must have landed before the CTA's shared memory is released.
    mbar_wait_drain(BAR(B_QFULL), 0);
    if (kdone > 0) mbar_wait_drain(BAR(B_KFULL), (kdone - 1) & 1);
    if (vdone > 0) mbar_wait_drain(BAR(B_VFULL), (vdone - 1) & 1);
  } else if (warp == 9) {
    if (nt > 0) {
      // ================= MMA issuer =================
      constexpr uint32_t IDESC_QK = make_idesc(BN, false);
      constexpr uint32_t IDESC_PV = make_idesc(D, true);
      auto issue_qk = [&]() {  // S = Q . K_j^T
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint64_t ad = make_desc(sQ + (ks / 4) * (QBM * 128) + (ks % 4) * 32, 16, 1024);
          const uint64_t bd = make_desc(sK + (ks / 4) * (BN * 128) + (ks % 4) * 32, 16, 1024);
          umma_ss(tmem + QTM1_S, ad, bd, IDESC_QK, ks > 0 ? 1u : 0u);
        }
        umma_commit(BAR(B_SFULL));
        umma_commit(BAR(B_KEMPTY));
      };
      auto issue_pv = [&](int j, int part) {  // O += P . V_j, keys 64*part .. 64*part + 63
        constexpr int HALF = BN / 32;
#pragma unroll
        for (int u = 0; u < HALF; ++u) {
          const int ks = part * HALF + u;
          const uint64_t bd = make_desc(sV + ks * 2048, BN * 128, 1024);
          umma_ts(tmem + QTM1_O, tmem + QTM1_S + ks * 8, bd, IDESC_PV, (j > 0 || part > 0 || u > 0) ? 1u : 0u);
        }
        if (part == 1) {
          umma_commit(BAR(B_ODONE));
          umma_commit(BAR(B_VEMPTY));
        }
      };
      do {
        if (!(ok = mbar_wait(BAR(B_QFULL), 0, status))) break;
        if (!(ok = mbar_wait(BAR(B_KFULL), 0, status))) break;
        tc_fence_after();
        issue_qk();
        for (int j = 0; j < nt && ok; ++j) {
          if (!(ok = mbar_wait(BAR(B_PFULL), j & 1, status))) break;
          if (!(ok = mbar_wait(BAR(B_VFULL), j & 1, status))) break;
          tc_fence_after();
          issue_pv(j, 0);
          if (!(ok = mbar_wait(BAR(B_PFULL + 1), j & 1, status))) break;
          tc_fence_after();
          issue_pv(j, 1);
          if (j + 1 < nt) {
            if (!(ok = mbar_wait(BAR(B_KFULL), (j + 1) & 1, status))) break;
            tc_fence_after();
            issue_qk();
          }
        }
      } while (false);
    }
  } else {
    // ================= softmax: 16 rows per warp, a row pair per quad of threads =================
    const int qd = warp & 3, hf = (warp >> 2) & 1;
    const int q4 = lane & 3;
    const int rowA = qd * 32 + hf * 16 + (lane >> 2);
    const uint32_t lane16 = (uint32_t)(qd * 32 + hf * 16) << 16;
    const uint32_t t_s = tmem + lane16 + QTM1_S;
    const uint32_t t_o = tmem + lane16 + QTM1_O;
    QuadRows st = {-INFINITY, -INFINITY, 0.f, 0.f};
    for (int j = 0; j < nt; ++j) {
      const bool masked = j >= jm;
      const int limA = masked ? rowA + tq0 + s.P - __ldg(indices + off + j) * BN - 2 * q4 : 0x7fffffff - 8;
      ok = quad_softmax_block<D, BN, SKIP>(t_s, t_o, BAR(B_SFULL), j & 1, BAR(B_ODONE), (j - 1) & 1, BAR(B_PFULL),
                                                  BAR(B_PFULL + 1), j == 0, masked, limA, scale_log2, skip_log2, lane,
                                                  status, st) && ok;
    }
    quad_epilogue_sums<D>(st, lsum, rowA, q4, 1 + qd);
    const int row = qd * 32 + lane;
    const float l_row = lsum[row];
    if (nt > 0) {
      ok = mbar_wait(BAR(B_ODONE), (nt - 1) & 1, status) && ok;
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      const int t_row = tq0 + row;
      const bool in_seq = t_row < s.Nq;
      constexpr int OH = D / 2;
      __nv_bfloat16* orow = out + (long long)h * s.os_h + (long long)t_row * s.os_t + hf * OH;
      if (nt == 0) {
        for (int c = 0; c < OH / 8 && in_seq; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
      } else {
        tc_fence_after();
        const float inv = l_row > 0.f ? 1.0f / l_row : 0.f;
        const uint32_t t_o32 = tmem + ((uint32_t)(qd * 32) << 16) + QTM1_O + hf * OH;
#pragma unroll
        for (int c = 0; c < OH / 32; ++c) {
          uint32_t o[32];
          tmem_ld32(t_o32 + c * 32, o);
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
  if (warp == 8 && nt > 0) {
    tc_fence_after();
    tmem_dealloc(tmem, QTM1_COLS);
  }
}

// ------------------------------------------------------------------------------------------------
// Persistent form
// ------------------------------------------------------------------------------------------------
constexpr int QREC = 4;  // records in flight
enum { R_VALID = 0, R_H = 1, R_Q0 = 2, R_OFF = 3, R_N0 = 4, R_N1 = 5, R_JM0 = 6, R_JM1 = 7 };

template <int D, int BN, int NSLOT, bool SKIP>
__global__ void __maxnreg__(96)
sparse_attention_quad_persistent_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                                        const __grid_constant__ CUtensorMap tmv, __nv_bfloat16* __restrict__ out,
                                        const int* __restrict__ items, const int* __restrict__ indices,
                                        int* __restrict__ status, int* __restrict__ sched, Shape s, float scale_log2,
                                        float skip_log2, int n_items) {
  using L = QuadSmem<D, BN, NSLOT>;
  static_assert(BN == 128 && D == 128, "the quad-layout kernels are written for head_dim 128 and 128-wide key blocks");
  extern __shared__ unsigned char att_smem_raw[];

  const uint32_t raw = smem_u32(att_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gbase = att_smem_raw + (base - raw);
  const uint32_t sQ = base + L::OFF_Q, sRing = base + L::OFF_RING;
  float* lsum = reinterpret_cast<float*>(gbase + L::OFF_LSUM);
  volatile int* rec = reinterpret_cast<volatile int*>(gbase + L::OFF_REC);
  const uint32_t bar0 = base + L::OFF_BAR;
  auto BAR = [&](int i) { return bar0 + 8u * i; };
  const int B_QFULL = 0, B_QEMPTY = 2, B_FULL = 4, B_EMPTY = 4 + NSLOT, B_SFULL = 4 + 2 * NSLOT, B_PFULL = B_SFULL + 2,
            B_ODONE = B_PFULL + 4, B_OREAD = B_ODONE + 2, B_RFULL = B_OREAD + 2, B_REMPTY = B_RFULL + QREC;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gbase + L::OFF_BAR + L::NBAR * 8);

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);

  if (warp == 16) {
    if (lane == 0) {
      for (int t = 0; t < 2; ++t) {
        mbar_init(BAR(B_QFULL + t), 1);
        mbar_init(BAR(B_QEMPTY + t), 1);
        mbar_init(BAR(B_SFULL + t), 1);
        mbar_init(BAR(B_PFULL + 2 * t), 8);
        mbar_init(BAR(B_PFULL + 2 * t + 1), 8);
        mbar_init(BAR(B_ODONE + t), 1);
        mbar_init(BAR(B_OREAD + t), 8);  // the tile's softmax warps have read O out of tensor memory
      }
      for (int t = 0; t < NSLOT; ++t) {
        mbar_init(BAR(B_FULL + t), 1);
        mbar_init(BAR(B_EMPTY + t), 1);
      }
      for (int t = 0; t < QREC; ++t) {
        mbar_init(BAR(B_RFULL + t), 1);
        mbar_init(BAR(B_REMPTY + t), 18);  // producer, MMA warp and the 16 softmax warps
      }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      fence_async_smem();
    }
    __syncwarp();
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), QTM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  bool ok = true;
  const int pairs_per_seg = s.L_S / (2 * QBM);

  // a reader's view of record kk: waits until it is published, copies what it needs, releases the slot
  auto rec_wait = [&](int kk) {
    bool w = mbar_wait(BAR(B_RFULL + kk % QREC), (kk / QREC) & 1, status);
    return __all_sync(0xffffffffu, w);
  };
  auto rec_release = [&](int kk) {
    __syncwarp();
    if (lane == 0) mbar_arrive(BAR(B_REMPTY + kk % QREC));
  };

  if (warp == 18) {
    // ================= scheduler: items off the global counter, block-list look-up, record ring =================
    // an earlier launch gave up: take no work (one answer for the warp, whatever the lanes read)
    const bool dead = __any_sync(0xffffffffu, *reinterpret_cast<volatile int*>(status) != 0);
    for (int kk = 0;; ++kk) {
      int item = n_items;
      if (!dead && ok) {
        if (lane == 0) item = atomicAdd(sched, 1);
        item = __shfl_sync(0xffffffffu, item, 0);
      }
      const bool valid = item < n_items;
      int h = 0, q0 = 0, off = 0, n0 = 0, n1 = 0, jm0 = 0, jm1 = 0;
      if (valid) {
        int bid = item;
        const int pr = bid % pairs_per_seg;
        bid /= pairs_per_seg;
        h = bid % s.H;
        const int i = s.C_S - 1 - bid / s.H;  // long lists (late segments) first
        const long long cell = (long long)(h / s.list_div) * s.C_S + i;
        q0 = i * s.L_S + pr * 2 * QBM;
        const int4* recp = reinterpret_cast<const int4*>(items + (cell * pairs_per_seg + pr) * 8);
        const int4 r0 = __ldg(recp), r1 = __ldg(recp + 1);  // (a pair beyond the sequence has n0 = n1 = 0 and stores nothing)
        off = r0.x;
        n0 = r0.y;
        n1 = r0.z;
        jm0 = r0.w;
        jm1 = r1.x;
      }
      {  // record kk - QREC has been read?  (polled at leisure: the ring is four records deep, and a spinning warp
         //  would take issue slots from the softmax warps of its SM sub-partition)
        const uint32_t bar = BAR(B_REMPTY + kk % QREC), par = ((kk / QREC) & 1) ^ 1;
        const long long t0 = clock64();
        while (ok && !mbar_try_wait(bar, par)) {
          __nanosleep(2000);
          if (*reinterpret_cast<volatile int*>(status) != 0) ok = false;
          else if (clock64() - t0 > (1LL << 30)) {
            atomicExch(status, (int)EI_ERR_DEVICE_TIMEOUT);
            ok = false;
          }
        }
      }
      ok = __all_sync(0xffffffffu, ok);
      if (lane == 0) {
        volatile int* r = rec + (kk % QREC) * 8;
        r[R_VALID] = (valid && ok) ? 1 : 0;
        r[R_H] = h;
        r[R_Q0] = q0;
        r[R_OFF] = off;
        r[R_N0] = n0;
        r[R_N1] = n1;
        r[R_JM0] = jm0;
        r[R_JM1] = jm1;
        __threadfence_block();
        mbar_arrive(BAR(B_RFULL + kk % QREC));
      }
      __syncwarp();
      if (!valid || !ok) break;
    }
  } else if (warp == 16) {
    // ================= TMA producer =================
    int ucount = 0;   // ring items issued so far, over all work items
    int last_q = -1;  // the last item whose Q tiles were loaded
    auto ring_load = [&](int blk, int g, bool is_v) -> bool {
      const int slot = ucount % NSLOT;
      if (!mbar_wait(BAR(B_EMPTY + slot), ((ucount / NSLOT) & 1) ^ 1, status)) return false;
      mbar_expect_tx(BAR(B_FULL + slot), L::KV_BYTES);
      const CUtensorMap* tm = is_v ? &tmv : &tmk;
#pragma unroll
      for (int p = 0; p < D / 64; ++p)
        tma_load_3d(sRing + slot * L::KV_BYTES + p * (BN * 128), tm, p * 64, blk * BN, g, BAR(B_FULL + slot));
      ++ucount;
      return true;
    };
    for (int kk = 0;; ++kk) {
      ok = rec_wait(kk) && ok;
      const volatile int* r = rec + (kk % QREC) * 8;
      const int valid = ok ? r[R_VALID] : 0, h = r[R_H], q0 = r[R_Q0], off = r[R_OFF], n1 = r[R_N1];
      rec_release(kk);
      if (!valid) break;
      const int g = h / s.G;
      // K_0 first (it only needs a ring slot), then the Q tiles as the previous item's last Q.K^T let go of them
      int blk = n1 > 0 ? __ldg(indices + off) : 0;
      if (n1 > 0 && !(ok = ring_load(blk, g, false))) break;
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        ok = mbar_wait(BAR(B_QEMPTY + t), (kk & 1) ^ 1, status);
        if (!ok) break;
        mbar_expect_tx(BAR(B_QFULL + t), L::Q_BYTES);
#pragma unroll
        for (int p = 0; p < D / 64; ++p)
          tma_load_3d(sQ + t * L::Q_BYTES + p * (QBM * 128), &tmq, p * 64, q0 + t * QBM, h, BAR(B_QFULL + t));
      }
      if (!ok) break;
      last_q = kk;
      for (int u = 1; u < 2 * n1; ++u) {
        const int blk_next = ((u & 1) && (u >> 1) + 1 < n1) ? __ldg(indices + off + (u >> 1) + 1) : blk;
        if (!(ok = ring_load(blk, g, (u & 1) != 0))) break;
        blk = blk_next;
      }
      if (!ok) break;
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
    int itc[2] = {0, 0};  // blocks issued per tile over all items (parity of p_full)
    auto wait_ring = [&](int u) { return mbar_wait(BAR(B_FULL + u % NSLOT), (u / NSLOT) & 1, status); };
    for (int kk = 0;; ++kk) {
      ok = rec_wait(kk) && ok;
      const volatile int* r = rec + (kk % QREC) * 8;
      const int valid = ok ? r[R_VALID] : 0, n0 = r[R_N0], n1 = r[R_N1];
      rec_release(kk);
      if (!valid) break;
      const int nn[2] = {n0, n1};
      auto issue_qk = [&](int t, int j) {  // S_t = Q_t . K_j^T ; the item's last one also releases Q_t
        const uint32_t kbase = sRing + ((ubase + 2 * j) % NSLOT) * L::KV_BYTES;
        const uint32_t qbase = sQ + t * L::Q_BYTES;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint64_t ad = make_desc(qbase + (ks / 4) * (QBM * 128) + (ks % 4) * 32, 16, 1024);
          const uint64_t bd = make_desc(kbase + (ks / 4) * (BN * 128) + (ks % 4) * 32, 16, 1024);
          umma_ss(tmem + qtm_s(t), ad, bd, IDESC_QK, ks > 0 ? 1u : 0u);
        }
        umma_commit(BAR(B_SFULL + t));
        if (j == nn[t] - 1) umma_commit(BAR(B_QEMPTY + t));
      };
      auto issue_pv = [&](int t, int j, int part) {
        const uint32_t vbase = sRing + ((ubase + 2 * j + 1) % NSLOT) * L::KV_BYTES;
        constexpr int HALF = BN / 32;
#pragma unroll
        for (int u = 0; u < HALF; ++u) {
          const int ks = part * HALF + u;
          const uint64_t bd = make_desc(vbase + ks * 2048, BN * 128, 1024);
          umma_ts(tmem + qtm_o(t), tmem + qtm_s(t) + ks * 8, bd, IDESC_PV, (j > 0 || part > 0 || u > 0) ? 1u : 0u);
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
            if (j == 0 && !(ok = mbar_wait(BAR(B_OREAD), (kk & 1) ^ 1, status))) break;  // the previous O_0 has been read
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
          if (j == 0 && !(ok = mbar_wait(BAR(B_OREAD + 1), (kk & 1) ^ 1, status))) break;
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
    // ================= softmax: tile t = warp / 8, 16 rows per warp, a row pair per quad of threads =================
    // (after a timed-out wait the threads keep going through the motions -- later waits return at once -- so that
    //  both warps of a quadrant reach the same named barriers)
    const int t = warp >> 3;
    const int qd = warp & 3, hf = (warp >> 2) & 1;
    const int q4 = lane & 3;
    const int rowA = qd * 32 + hf * 16 + (lane >> 2);
    const uint32_t lane16 = (uint32_t)(qd * 32 + hf * 16) << 16;
    const uint32_t t_s = tmem + lane16 + qtm_s(t);
    const uint32_t t_o = tmem + lane16 + qtm_o(t);
    const int row = qd * 32 + lane;
    constexpr int OH = D / 2;
    const uint32_t t_o32 = tmem + ((uint32_t)(qd * 32) << 16) + qtm_o(t) + hf * OH;
    int itc = 0;  // blocks of my tile over all items (parity of s_full / o_done)
    for (int kk = 0;; ++kk) {
      ok = rec_wait(kk) && ok;
      const volatile int* r = rec + (kk % QREC) * 8;
      const int valid = ok ? r[R_VALID] : 0, h = r[R_H], q0 = r[R_Q0], off = r[R_OFF];
      const int nt = t ? r[R_N1] : r[R_N0];
      const int jm = t ? r[R_JM1] : r[R_JM0];
      rec_release(kk);
      if (!valid) break;
      const int tq0 = q0 + t * QBM;
      QuadRows st = {-INFINITY, -INFINITY, 0.f, 0.f};
      for (int j = 0; j < nt; ++j, ++itc) {
        const bool masked = j >= jm;
        const int limA = masked ? rowA + tq0 + s.P - __ldg(indices + off + j) * BN - 2 * q4 : 0x7fffffff - 8;
        ok = quad_softmax_block<D, BN, SKIP>(t_s, t_o, BAR(B_SFULL + t), itc & 1, BAR(B_ODONE + t), (itc - 1) & 1,
                                              BAR(B_PFULL + 2 * t), BAR(B_PFULL + 2 * t + 1), j == 0, masked, limA,
                                              scale_log2, skip_log2, lane, status, st) && ok;
      }
      float* ls = lsum + t * QBM;
      quad_epilogue_sums<D>(st, ls, rowA, q4, 1 + t * 4 + qd);
      const float l_row = ls[row];
      asm volatile("bar.sync %0, %1;" ::"r"(1 + t * 4 + qd), "r"(64) : "memory");  // both warps have read: the cells may be written again
      const int t_row = tq0 + row;
      const bool in_seq = t_row < s.Nq;  // rows beyond the sequence join the warp-wide loads, only their stores are dropped
      __nv_bfloat16* orow = out + (long long)h * s.os_h + (long long)t_row * s.os_t + hf * OH;
      if (nt == 0) {
        if (lane == 0) mbar_arrive(BAR(B_OREAD + t));  // keeps the barrier's phase in step with the item count
        for (int c = 0; c < OH / 8 && in_seq; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
        continue;
      }
      ok = mbar_wait(BAR(B_ODONE + t), (itc - 1) & 1, status) && ok;
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      const float inv = l_row > 0.f ? 1.0f / l_row : 0.f;
      quad_store_rows<D / 2>(t_o32, orow, inv, in_seq && ok, BAR(B_OREAD + t), lane);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 16) {
    tc_fence_after();
    tmem_dealloc(tmem, QTM_COLS);
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
// Per-item records.  What a CTA needs to know about its (list head, segment, tile pair) before it can start --
// where the block list is, how many of its blocks each of the two tiles sees at all, from which entry on they
// need the causal mask, and the first block -- is a function of the plan alone, so it is worked out once per
// plan (one warp per record) instead of by every CTA through a chain of dependent global loads.
// Record (8 ints): list offset, n0, n1, jm0, jm1, first block, 0, 0.
// ------------------------------------------------------------------------------------------------
__global__ void attention_items_kernel(const int* __restrict__ offsets, const int* __restrict__ indices,
                                       int* __restrict__ items, Shape s, long long n_rec, int pairs_per_seg) {
  const long long rec = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (rec >= n_rec) return;
  const long long cell = rec / pairs_per_seg;
  const int off = __ldg(offsets + cell);
  attention_item_record(s, (int)(cell % s.C_S), (int)(rec % pairs_per_seg), off, __ldg(offsets + cell + 1) - off,
                        indices + off, items + rec * 8, lane);
}

cudaError_t launch_attention_items(const Shape& ls, const int* offsets, const int* indices, int* items, cudaStream_t st) {
  if (ls.L_S % (2 * QBM) != 0) return cudaSuccess;  // shapes the tile-pair kernels do not take
  const int pairs = ls.L_S / (2 * QBM);
  const long long n_rec = ls.cells * pairs;
  if (n_rec == 0) return cudaSuccess;
  attention_items_kernel<<<(unsigned)((n_rec + 3) / 4), 128, 0, st>>>(offsets, indices, items, ls, n_rec, pairs);
  return cudaGetLastError();
}

// One launch over the sequences of a packed batch: the tensor maps span the whole packed tensors (n_tokens rows),
// a CTA adds its sequence's first token to the row coordinates.  What lies behind a sequence's last row is the next
// sequence's data instead of the zero fill a tensor's end gives: queries there are computed and not stored, keys
// there lie above every row of the sequence and fall to the causal mask, their V rows meet P = 0.
int launch_attention_quad_packed(const PackedSeq* pk, const PackedSeq* pk_host, int npk, long long n_tokens,
                                 const AttnArgs& a, cudaStream_t st) {
  constexpr int D = 128, BN = 128, NSLOT = 5;
  using L = QuadSmem<D, BN, NSLOT>;
  const Shape& s = pk_host[npk - 1].s;
  if (!a.items || n_tokens <= 0) return EI_ERR_INVALID_ARG;
  CUtensorMap tmq, tmk, tmv;
  if (!make_tensor_map(&tmq, a.q, D, (int)n_tokens, s.H, s.qs_t, s.qs_h, QBM) ||
      !make_tensor_map(&tmk, a.k, D, (int)n_tokens, s.Hkv, s.ks_t, s.ks_h, BN) ||
      !make_tensor_map(&tmv, a.v, D, (int)n_tokens, s.Hkv, s.vs_t, s.vs_h, BN))
    return EI_ERR_CUDA;
  const long long grid = pk_host[npk - 1].w_att + (long long)s.H * s.C_S * (s.L_S / (2 * QBM));
  const float scale_log2 = a.scale * 1.4426950408889634f;
  const bool skip = a.skip_log2 < INFINITY;
  auto kern = skip ? sparse_attention_quad_kernel<D, BN, NSLOT, true> : sparse_attention_quad_kernel<D, BN, NSLOT, false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES) != cudaSuccess)
    return EI_ERR_CUDA;
  kern<<<(unsigned)grid, QUAD_THREADS, L::DYN_BYTES, st>>>(tmq, tmk, tmv, a.out, a.items, a.indices, a.status, s, scale_log2,
                                                          a.skip_log2, pk, npk);
  return cudaGetLastError() == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

int launch_attention_quad(const Shape& s, const AttnArgs& a, cudaStream_t st) {
  constexpr int D = 128, BN = 128, NSLOT = 5;
  using L = QuadSmem<D, BN, NSLOT>;
  static_assert(L::DYN_BYTES <= 232448, "shared memory budget exceeded");
  if (!a.items) return EI_ERR_INVALID_ARG;
  CUtensorMap tmq, tmk, tmv;
  if (!make_tensor_map(&tmq, a.q, D, s.Nq, s.H, s.qs_t, s.qs_h, QBM) ||
      !make_tensor_map(&tmk, a.k, D, s.N, s.Hkv, s.ks_t, s.ks_h, BN) ||
      !make_tensor_map(&tmv, a.v, D, s.N, s.Hkv, s.vs_t, s.vs_h, BN))
    return EI_ERR_CUDA;
  const long long n_items = (long long)s.H * s.C_S * (s.L_S / (2 * QBM));
  const float scale_log2 = a.scale * 1.4426950408889634f;
  const bool skip = a.skip_log2 < INFINITY;  // the shortcut for negligible rows is compiled in only where it is asked for
  if (a.persistent && a.sched) {
    auto kern = skip ? sparse_attention_quad_persistent_kernel<D, BN, NSLOT, true>
                     : sparse_attention_quad_persistent_kernel<D, BN, NSLOT, false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES) != cudaSuccess)
      return EI_ERR_CUDA;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const unsigned grid = (unsigned)(n_items < sms ? n_items : sms);  // one CTA per SM; items come off a counter
    kern<<<grid, QUADP_THREADS, L::DYN_BYTES, st>>>(tmq, tmk, tmv, a.out, a.items, a.indices, a.status, a.sched, s,
                                                  scale_log2, a.skip_log2, (int)n_items);
  } else if (a.single_tile) {
    using L1 = Quad1Smem<D, BN>;
    static_assert(2 * (L1::DYN_BYTES + 1024) <= 233472, "two CTAs must fit the shared memory of an SM");
    auto kern = skip ? sparse_attention_quad1_kernel<D, BN, true> : sparse_attention_quad1_kernel<D, BN, false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L1::DYN_BYTES) != cudaSuccess)
      return EI_ERR_CUDA;
    kern<<<(unsigned)(2 * n_items), QUAD1_THREADS, L1::DYN_BYTES, st>>>(tmq, tmk, tmv, a.out, a.items, a.indices, a.status, s,
                                                                     scale_log2, a.skip_log2);
  } else {
    auto kern = skip ? sparse_attention_quad_kernel<D, BN, NSLOT, true> : sparse_attention_quad_kernel<D, BN, NSLOT, false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES) != cudaSuccess)
      return EI_ERR_CUDA;
    kern<<<(unsigned)n_items, QUAD_THREADS, L::DYN_BYTES, st>>>(tmq, tmk, tmv, a.out, a.items, a.indices, a.status, s,
                                                               scale_log2, a.skip_log2, nullptr, 0);
  }
  return cudaGetLastError() == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

}  // namespace ei
