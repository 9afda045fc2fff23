// Stage 4, three-buffer kernel: causal GQA flash attention over the selected key blocks (Eq. t_spa) for
// head_dim 128 and 128-wide key blocks, hand-written for sm_100a.
//
// The two-tile kernels keep S0, S1, O0, O1 in the 512 tensor-memory columns, so every tile has ONE S buffer and a
// key block goes round Q.K^T -> softmax -> P.V before the next Q.K^T of that tile can be issued: two blocks are
// in flight per SM and the length of that round trip, not any one unit, bounds the kernel.  Here a CTA works on
// ONE 128-row query tile at a time with THREE S buffers and one O (3 x 128 + 128 columns): Q.K^T runs three key
// blocks ahead of P.V, and the sixteen softmax warps form two sets that take alternate key blocks, so that a
// block's logits are already in tensor memory when a set turns to it.
//
//   warps 0-7   set 0: key blocks J = 0, 2, 4, ... (J counts the CTA's blocks across its tiles)
//   warps 8-15  set 1: J = 1, 3, 5, ...
//                within a set warp w owns lanes 32*(w%4) + 16*((w/4)%2) .. +15: sixteen query rows and all 128
//                key columns through the 16-lane tensor-memory shapes (a row pair per quad of threads)
//   warp 16     TMA producer (Q double-buffered, K ring, V ring)    warp 17   Q.K^T issuer    warp 18   P.V issuer
//
// The online softmax of a row is sequential in the key blocks only through its reference maximum (O is rescaled
// lazily, when the maximum grew by more than 2^8).  The warp of set 0 and the warp of set 1 that own the same
// rows pass that reference back and forth: after the row maxima of block J are known -- long before its
// exponentials are done -- the owner publishes the reference valid from block J on in shared memory and arrives
// on an mbarrier; the other set's warp picks it up when it has the maxima of block J+1.  Either set keeps its own
// partial row sums, brought to the current reference when it changes; they are added in the tile's epilogue.
// A CTA takes several consecutive tiles of a (head, segment) cell: the block stream runs on across the tile
// boundary (Q.K^T of the next tile's first blocks is issued while the previous tile's last blocks are still in
// the softmax), only the first P.V of a tile waits until the previous tile's O has been read out.
// Every mbarrier wait is bounded; on expiry the status word is set, later waits return at once, and the CTA
// drains its loads and frees its tensor memory.
#include <cuda.h>

#include "ei_internal.cuh"
#include "ei_sm100.cuh"

namespace ei {

constexpr int TRI_THREADS = 608;
constexpr int TBM = 128;
constexpr int TRI_NK = 2, TRI_NV = 2;  // K and V ring slots
constexpr int TRI_MAXT = 8;            // tiles per CTA at most
constexpr float TRI_RESCALE_THRESHOLD = 8.0f;  // log2 units
__host__ __device__ constexpr uint32_t ttm_s(int b) { return 128u * (uint32_t)b; }
constexpr uint32_t TTM_O = 384, TTM_COLS = 512;

namespace tri {
// 16 lanes x 64 columns of fp32: r[4i + {0,1}] = row t/4, columns 8i + 2(t%4) + {0,1}; r[4i + {2,3}] = row t/4 + 8
__device__ __forceinline__ void ld_16x64(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// 16 lanes x 32 packed columns (64 bf16): r[2i] = row t/4, packed column 4i + t%4; r[2i + 1] = row t/4 + 8
__device__ __forceinline__ void st_16x32(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.16x128b.x8.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
      ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void ld_16x8(uint32_t taddr, uint32_t (&r)[4]) {
  asm volatile("tcgen05.ld.sync.aligned.16x256b.x1.b32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void st_16x8(uint32_t taddr, const uint32_t (&r)[4]) {
  asm volatile("tcgen05.st.sync.aligned.16x256b.x1.b32 [%4], {%0,%1,%2,%3};" ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]),
               "r"(taddr)
               : "memory");
}

// running state of a thread's two query rows: the reference maxima its sums are relative to (raw logit units)
// and this set's partial row sums
struct Rows {
  float mrA, mrB, lA, lB;
};

// O[my two rows, all columns] *= alpha, once the P.V products issued so far have landed (rare: only when a row's
// maximum moved by more than 2^8).  Out of line: its registers and loop stay out of the softmax loop.
template <int D>
__device__ __noinline__ bool rescale(uint32_t t_o, float alA, float alB, uint32_t bar_odone, uint32_t par, int* status) {
  bool ok = mbar_wait(bar_odone, par, status);
  ok = __all_sync(0xffffffffu, ok);
  tc_fence_after();
#pragma unroll 1
  for (int c = 0; c < D / 8; ++c) {  // eight columns at a time
    uint32_t o[4];
    ld_16x8(t_o + c * 8, o);
    tmem_wait_ld();
    o[0] = __float_as_uint(__uint_as_float(o[0]) * alA);
    o[1] = __float_as_uint(__uint_as_float(o[1]) * alA);
    o[2] = __float_as_uint(__uint_as_float(o[2]) * alB);
    o[3] = __float_as_uint(__uint_as_float(o[3]) * alB);
    st_16x8(t_o + c * 8, o);
  }
  tmem_wait_st();
  return ok;
}

// my partial sum, relative to reference `from`, brought to reference `to` (a sum of zero stays zero whatever the
// references are: -inf before the first block)
__device__ __forceinline__ float realign(float l, float from, float to, float scale_log2) {
  return (l == 0.f || from == to) ? l : l * fast_ex2((from - to) * scale_log2);
}

// One key block of the online softmax for the 16 rows of a warp.
//   first:    the tile's first block (the references are taken from it, O holds nothing yet)
//   J:        the block's number in the CTA's stream (odd / even decides the set; J - 1 is the other set's)
//   limA:     causal bound for row A in units of my column offsets: key column c of the block is visible to row A
//             iff c - 2*(lane%4) <= limA, to row B iff <= limA + 8
template <int D, int BN, bool SKIP>
__device__ __forceinline__ bool softmax_block(uint32_t t_s, uint32_t t_o, uint32_t bar_sfull, uint32_t par_sfull,
                                              uint32_t bar_odone, uint32_t par_odone_prev, uint32_t bar_p0,
                                              uint32_t bar_p1, uint32_t bar_mx_mine, uint32_t bar_mx_other,
                                              uint32_t par_mx_other, float* mref_mine, const volatile float* mref_other,
                                              bool first, bool masked, int limA, float scale_log2, float skip_log2,
                                              int lane, int* status, Rows& st) {
  bool ok = mbar_wait(bar_sfull, par_sfull, status);
  ok = __all_sync(0xffffffffu, ok);
  tc_fence_after();
  uint32_t xa[32], xb[32];  // columns 0..63 and 64..127: [4i + {0,1}] row A, [4i + {2,3}] row B, columns 8i + 2*(lane%4) + {0,1}
  ld_16x64(t_s, xa);
  ld_16x64(t_s + 64, xb);
  tmem_wait_ld();  // (nothing that may call a function between the loads and this wait: the loads land in the
                   //  registers asynchronously, and a call could save and restore them in between)
  // the reference valid after block J - 1, from the warp of the other set that owns my rows
  float pmA = 0.f, pmB = 0.f;
  if (!first) {
    ok = mbar_wait(bar_mx_other, par_mx_other, status) && ok;
    pmA = mref_other[lane >> 2];
    pmB = mref_other[(lane >> 2) + 8];
  }
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
  float alA = 1.0f, alB = 1.0f;
  bool any_need = false;
  if (first) {
    st.mrA = lmA;
    st.mrB = lmB;
  } else {
    // (the exponentials of the rare cases sit behind ONE warp-uniform branch: on the special-function unit they
    //  would queue behind the other warps' probabilities, on the path every block takes)
    const bool needA = (lmA - pmA) * scale_log2 > TRI_RESCALE_THRESHOLD;  // a reference of -inf: inf > 8
    const bool needB = (lmB - pmB) * scale_log2 > TRI_RESCALE_THRESHOLD;
    const bool moved = st.mrA != pmA || st.mrB != pmB;  // the other set moved a reference
    if (__any_sync(0xffffffffu, needA || needB || moved)) {
      st.lA = realign(st.lA, st.mrA, pmA, scale_log2);
      st.lB = realign(st.lB, st.mrB, pmB, scale_log2);
      if (needA) alA = fast_ex2((pmA - lmA) * scale_log2);
      if (needB) alB = fast_ex2((pmB - lmB) * scale_log2);
      any_need = __any_sync(0xffffffffu, needA || needB);
    }
    st.mrA = needA ? lmA : pmA;
    st.mrB = needB ? lmB : pmB;
  }
  // publish the reference valid from this block on, before the exponentials: the other set needs nothing else
  if ((lane & 3) == 0) {
    mref_mine[lane >> 2] = st.mrA;
    mref_mine[(lane >> 2) + 8] = st.mrB;
  }
  __syncwarp();
  if (lane == 0) mbar_arrive(bar_mx_mine);
  if (any_need) {
    ok = rescale<D>(t_o, alA, alB, bar_odone, par_odone_prev, status) && ok;
    st.lA *= alA;
    st.lB *= alB;
  }
  // Rows whose largest logit lies more than skip_log2 binary orders below the reference maximum hold only terms
  // below 2^-skip_log2 of the row's largest: where that is so for all 16 rows of the warp, P is zero and nothing
  // is exponentiated.  (A fully masked row, -inf, qualifies; a reference of -inf gives NaN: not.)
  if (SKIP && __all_sync(0xffffffffu,
                         (lmA - st.mrA) * scale_log2 < -skip_log2 && (lmB - st.mrB) * scale_log2 < -skip_log2)) {
    uint32_t(&zero)[16] = *reinterpret_cast<uint32_t(*)[16]>(&xa[0]);
#pragma unroll
    for (int e = 0; e < 16; ++e) zero[e] = 0u;
    st_16x32(t_s, zero);
    st_16x32(t_s + 32, zero);
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
  // pair e of a half goes back into register e of that half's own array (its inputs 2e, 2e+1 are read before).
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
    st_16x32(t_s + part * 32, *reinterpret_cast<uint32_t(*)[16]>(&x[0]));
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
}  // namespace tri

template <int D, int BN>
struct TriSmem {
  static constexpr int Q_BYTES = TBM * D * 2;
  static constexpr int KV_BYTES = BN * D * 2;
  static constexpr int OFF_Q = 0;  // two buffers
  static constexpr int OFF_K = 2 * Q_BYTES;
  static constexpr int OFF_V = OFF_K + TRI_NK * KV_BYTES;
  static constexpr int OFF_LSUM = OFF_V + TRI_NV * KV_BYTES;  // float [tile parity][set][128 rows]
  static constexpr int OFF_MREF = OFF_LSUM + 2 * 2 * TBM * 4;  // float [set][128 rows]
  static constexpr int OFF_TILE = OFF_MREF + 2 * TBM * 4;      // int [MAXT][2] (blocks, first masked entry) + [4] (off, blk0, ta, tb)
  static constexpr int OFF_BAR = OFF_TILE + TRI_MAXT * 8 + 16;
  // q_full[2] q_empty[2] k_full/k_empty v_full/v_empty s_full[3] p_full[3][2] o_done[3] o_read mx[2][8]
  static constexpr int NBAR = 4 + 2 * TRI_NK + 2 * TRI_NV + 3 + 6 + 3 + 1 + 16 + 3;
  static constexpr int TOTAL = OFF_BAR + NBAR * 8 + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;
};

template <int D, int BN, bool SKIP>
__global__ void __maxnreg__(96)
sparse_attention_tri_kernel(const __grid_constant__ CUtensorMap tmq, const __grid_constant__ CUtensorMap tmk,
                            const __grid_constant__ CUtensorMap tmv, __nv_bfloat16* __restrict__ out,
                            const int* __restrict__ items, const int* __restrict__ indices, int* __restrict__ status,
                            Shape s, float scale_log2, float skip_log2, int NT) {
  using L = TriSmem<D, BN>;
  static_assert(BN == 128 && D == 128, "the three-buffer kernel is written for head_dim 128 and 128-wide key blocks");
  extern __shared__ unsigned char att_smem_raw[];

  const uint32_t raw = smem_u32(att_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* gbase = att_smem_raw + (base - raw);
  const uint32_t sQ = base + L::OFF_Q, sK = base + L::OFF_K, sV = base + L::OFF_V;
  float* lsum = reinterpret_cast<float*>(gbase + L::OFF_LSUM);
  float* mref = reinterpret_cast<float*>(gbase + L::OFF_MREF);
  volatile int* tinfo = reinterpret_cast<volatile int*>(gbase + L::OFF_TILE);
  const uint32_t bar0 = base + L::OFF_BAR;
  auto BAR = [&](int i) { return bar0 + 8u * i; };
  constexpr int B_QFULL = 0, B_QEMPTY = 2, B_KFULL = 4, B_KEMPTY = B_KFULL + TRI_NK, B_VFULL = B_KEMPTY + TRI_NK,
                B_VEMPTY = B_VFULL + TRI_NV, B_SFULL = B_VEMPTY + TRI_NV, B_PFULL = B_SFULL + 3, B_ODONE = B_PFULL + 6,
                B_OREAD = B_ODONE + 3, B_MX = B_OREAD + 1, B_PVISS = B_MX + 16;  // p_full: 2*buffer + part; o_done: buffer; mx: 8*set + warp
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gbase + L::OFF_BAR + L::NBAR * 8);

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);

  const int tiles_per_seg = s.L_S / TBM, pairs_per_seg = tiles_per_seg / 2, groups_per_seg = tiles_per_seg / NT;
  int bid = blockIdx.x;
  const int tile0 = (bid % groups_per_seg) * NT;  // my tiles: tile0 .. tile0 + NT - 1 of the segment
  bid /= groups_per_seg;
  const int h = bid % s.H;
  const int i = s.C_S - 1 - bid / s.H;  // long lists (late segments) first
  const int g = h / s.G;
  const long long cell = (long long)(h / s.list_div) * s.C_S + i;
  const int q00 = i * s.L_S + tile0 * TBM;
  if (q00 >= s.Nq) return;  // tiles of the short last segment that lie beyond the sequence (CTA-uniform)

  if (warp == 16) {
    if (lane == 0) {
      for (int t = 0; t < 2; ++t) {
        mbar_init(BAR(B_QFULL + t), 1);
        mbar_init(BAR(B_QEMPTY + t), 1);
      }
      for (int t = 0; t < TRI_NK; ++t) {
        mbar_init(BAR(B_KFULL + t), 1);
        mbar_init(BAR(B_KEMPTY + t), 1);
      }
      for (int t = 0; t < TRI_NV; ++t) {
        mbar_init(BAR(B_VFULL + t), 1);
        mbar_init(BAR(B_VEMPTY + t), 1);
      }
      for (int t = 0; t < 3; ++t) {
        mbar_init(BAR(B_SFULL + t), 1);
        mbar_init(BAR(B_PFULL + 2 * t), 8);  // one arrival per softmax warp of the set that has the block
        mbar_init(BAR(B_PFULL + 2 * t + 1), 8);
      }
      for (int t = 0; t < 3; ++t) mbar_init(BAR(B_ODONE + t), 1);
      mbar_init(BAR(B_OREAD), 16);
      for (int t = 0; t < 16; ++t) mbar_init(BAR(B_MX + t), 1);
      for (int t = 0; t < 3; ++t) mbar_init(BAR(B_PVISS + t), 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      fence_async_smem();
    }
    // tile table: blocks visible to each of my tiles and the first entry that needs the causal mask.  Tiles that
    // start beyond the sequence are left out; tiles that see no block at all (hand-made lists) come first, since
    // the number of visible blocks cannot fall from one tile to the next.
    int n = 0, jm = 0, off = 0, blk0 = 0;
    if (lane < NT && q00 + lane * TBM < s.Nq) {
      const int tt = tile0 + lane;
      const int4* recp = reinterpret_cast<const int4*>(items + (cell * pairs_per_seg + (tt >> 1)) * 8);
      const int4 r0 = __ldg(recp), r1 = __ldg(recp + 1);
      off = r0.x;
      n = (tt & 1) ? r0.z : r0.y;
      jm = (tt & 1) ? r1.x : r0.w;
      blk0 = r1.y;
    }
    const unsigned inseq = __ballot_sync(0xffffffffu, lane < NT && q00 + lane * TBM < s.Nq);
    const unsigned nonempty = __ballot_sync(0xffffffffu, n > 0);
    if (lane < TRI_MAXT) {
      tinfo[2 * lane] = n;
      tinfo[2 * lane + 1] = jm;
    }
    if (lane == 0) {
      tinfo[2 * TRI_MAXT + 0] = off;
      tinfo[2 * TRI_MAXT + 1] = blk0;
      tinfo[2 * TRI_MAXT + 2] = nonempty ? __ffs(nonempty) - 1 : __popc(inseq);  // ta: first tile with blocks
      tinfo[2 * TRI_MAXT + 3] = __popc(inseq);                                  // tb: tiles inside the sequence
    }
    __syncwarp();
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TTM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int off = tinfo[2 * TRI_MAXT], ta = tinfo[2 * TRI_MAXT + 2], tb = tinfo[2 * TRI_MAXT + 3];
  auto n_of = [&](int t) { return tinfo[2 * t]; };
  int total = 0;
  for (int t = ta; t < tb; ++t) total += n_of(t);

  bool ok = true;

  if (warp == 16) {
    // ================= TMA producer (whole warp, elected lane issues) =================
    auto load_q = [&](int t) {
      const int buf = (t - ta) & 1;
      mbar_expect_tx(BAR(B_QFULL + buf), L::Q_BYTES);
#pragma unroll
      for (int p = 0; p < D / 64; ++p)
        tma_load_3d(sQ + buf * L::Q_BYTES + p * (TBM * 128), &tmq, p * 64, q00 + t * TBM, h, BAR(B_QFULL + buf));
    };
    // block numbers of the list, 32 entries per coalesced load (a dependent global load per tile would put its
    // latency on every load issue): one register window for the K stream, one for the V stream
    const int nmax = tb > ta ? n_of(tb - 1) : 0;
    int kwin = -1, kreg = 0, vwin = -1, vreg = 0;
    auto entry = [&](int j, int& win, int& reg) {
      if ((j >> 5) != win) {
        win = j >> 5;
        reg = (win * 32 + lane < nmax) ? __ldg(indices + off + win * 32 + lane) : 0;
      }
      return __shfl_sync(0xffffffffu, reg, j & 31);
    };
    auto load_k = [&](int J, int j) {
      const int slot = J % TRI_NK, blk = entry(j, kwin, kreg);
      mbar_expect_tx(BAR(B_KFULL + slot), L::KV_BYTES);
#pragma unroll
      for (int p = 0; p < D / 64; ++p) tma_load_3d(sK + slot * L::KV_BYTES + p * (BN * 128), &tmk, p * 64, blk * BN, g, BAR(B_KFULL + slot));
    };
    auto load_v = [&](int J, int j) {
      const int slot = J % TRI_NV, blk = entry(j, vwin, vreg);
      mbar_expect_tx(BAR(B_VFULL + slot), L::KV_BYTES);
#pragma unroll
      for (int p = 0; p < D / 64; ++p) tma_load_3d(sV + slot * L::KV_BYTES + p * (BN * 128), &tmv, p * 64, blk * BN, g, BAR(B_VFULL + slot));
    };
    // The loads are issued in the order in which their slots come free.  P.V of block J is issued when the
    // softmax has finished block J; Q.K^T runs three blocks ahead of it, so K of block e can go into the slot
    // that Q.K^T of block e - 2 has read long before V of block e - 2 can go into the slot that P.V of block
    // e - 4 has read: K_e, then V_{e-2}, for e = 2, 3, ...; Q of the tile after next goes in when the first
    // Q.K^T of the following tile has completed (the one before it was the last to read the buffer).
    int kt = ta, kj = 0, vt = ta, vj = 0, ct = ta, cj = 0;  // (tile, entry) of the next K load, V load, and of block e - 2
    int nq = 0, nk = 0, nv = 0;                              // loads issued so far
    auto adv = [&](int& t, int& j) {
      if (++j >= n_of(t)) {
        j = 0;
        ++t;
      }
    };
    if (total > 0) {
      load_q(ta);
      nq = 1;
      if (ta + 1 < tb) {
        load_q(ta + 1);
        nq = 2;
      }
      for (; nk < TRI_NK && nk < total; ++nk) {
        load_k(nk, kj);
        adv(kt, kj);
      }
      for (; nv < TRI_NV && nv < total; ++nv) {
        load_v(nv, vj);
        adv(vt, vj);
      }
      static_assert(TRI_NK == 2 && TRI_NV == 2, "the issue order below is written for two K and two V slots");
      for (int e = 2; e < total + 2; ++e) {
        const int o = ct - ta;  // block e - 2 belongs to my o-th tile
        if (cj == 0 && o >= 1 && ct + 1 < tb) {
          ok = mbar_wait(BAR(B_QEMPTY + ((o - 1) & 1)), ((o - 1) >> 1) & 1, status);
          if (!ok) break;
          load_q(ct + 1);
          ++nq;
        }
        if (e < total) {
          ok = mbar_wait(BAR(B_KEMPTY + (e & 1)), ((e - 2) >> 1) & 1, status);
          if (!ok) break;
          load_k(e, kj);
          adv(kt, kj);
          ++nk;
        }
        if (e >= 4 && e - 2 < total) {
          ok = mbar_wait(BAR(B_VEMPTY + (e & 1)), ((e - 4) >> 1) & 1, status);
          if (!ok) break;
          load_v(e - 2, vj);
          adv(vt, vj);
          ++nv;
        }
        adv(ct, cj);
      }
      // Drain: every load issued here must have landed before the CTA's shared memory is released.
      for (int u = (nq > 2 ? nq - 2 : 0); u < nq; ++u) mbar_wait_drain(BAR(B_QFULL + (u & 1)), (u >> 1) & 1);
      for (int u = (nk > TRI_NK ? nk - TRI_NK : 0); u < nk; ++u) mbar_wait_drain(BAR(B_KFULL + u % TRI_NK), (u / TRI_NK) & 1);
      for (int u = (nv > TRI_NV ? nv - TRI_NV : 0); u < nv; ++u) mbar_wait_drain(BAR(B_VFULL + u % TRI_NV), (u / TRI_NV) & 1);
    }
  } else if (warp == 17) {
    // ================= Q.K^T issuer (whole warp, elected lane issues) =================
    // Two warps feed the tensor pipe: an issuing thread spends several hundred cycles per key block on waits,
    // fences, commits and bookkeeping around its MMAs, and while it does the pipe runs dry after the few
    // instructions it has queued; with the S = Q.K^T and the O += P.V streams in different warps one of them can
    // issue while the other is busy with its barriers.  The only order the two streams need is that Q.K^T of
    // block J + 3 must not overwrite the buffer P.V of block J reads P from: it is issued after that product has been
    // issued (the pipe executes in issue order; the hand-over is an mbarrier between tcgen05 fences).
    constexpr uint32_t IDESC_QK = make_idesc(BN, false);
    int qt = ta, qj = 0;
    for (int qJ = 0; qJ < total; ++qJ) {
      const int ord = qt - ta, nq = n_of(qt), b = qJ % 3;
      if (qj == 0 && !(ok = mbar_wait(BAR(B_QFULL + (ord & 1)), (ord >> 1) & 1, status))) break;
      if (!(ok = mbar_wait(BAR(B_KFULL + qJ % TRI_NK), (qJ / TRI_NK) & 1, status))) break;
      const uint32_t kbase = sK + (qJ % TRI_NK) * L::KV_BYTES, qbase = sQ + (ord & 1) * L::Q_BYTES;
      const uint64_t qdesc = make_desc(qbase, 16, 1024), kdesc = make_desc(kbase, 16, 1024);
      // (the operands first: once the buffer comes free nothing but the issue itself is left to do)
      if (qJ >= 3 && !(ok = mbar_wait(BAR(B_PVISS + b), ((qJ - 3) / 3) & 1, status))) break;
      tc_fence_after();
      umma_ss_d128(tmem + ttm_s(b), qdesc, kdesc, IDESC_QK);
      umma_commit(BAR(B_SFULL + b));
      umma_commit(BAR(B_KEMPTY + qJ % TRI_NK));
      if (qj == nq - 1) umma_commit(BAR(B_QEMPTY + (ord & 1)));
      if (++qj >= nq) {
        qj = 0;
        ++qt;
      }
    }
  } else if (warp == 18) {
    // ================= P.V issuer (whole warp, elected lane issues) =================
    constexpr uint32_t IDESC_PV = make_idesc(D, true);
    int pt = ta, pj = 0;
    for (int J = 0; J < total; ++J) {
      const int b = J % 3;
      const uint32_t par = (J / 3) & 1;
      const uint32_t vbase = sV + (J % TRI_NV) * L::KV_BYTES, a = tmem + ttm_s(b);
      // the previous tile's O must have been read out before this tile's first product overwrites it
      if (pj == 0 && pt > ta && !(ok = mbar_wait(BAR(B_OREAD), (pt - ta - 1) & 1, status))) break;
      if (!(ok = mbar_wait(BAR(B_PFULL + 2 * b), par, status))) break;
      if (!(ok = mbar_wait(BAR(B_VFULL + J % TRI_NV), (J / TRI_NV) & 1, status))) break;
      tc_fence_after();
      umma_ts_x4(tmem + TTM_O, a, make_desc(vbase, BN * 128, 1024), IDESC_PV, pj > 0 ? 1u : 0u);  // keys 0..63
      if (!(ok = mbar_wait(BAR(B_PFULL + 2 * b + 1), par, status))) break;
      tc_fence_after();
      umma_ts_x4(tmem + TTM_O, a + 32, make_desc(vbase + 8192, BN * 128, 1024), IDESC_PV, 1u);  // keys 64..127
      umma_commit(BAR(B_ODONE + b));
      umma_commit(BAR(B_VEMPTY + J % TRI_NV));
      tc_fence_before();  // P.V of this block is in the pipe: the Q.K^T that overwrites its P may be issued behind it
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_PVISS + b));
      if (++pj >= n_of(pt)) {
        pj = 0;
        ++pt;
      }
    }
  } else {
    // ================= softmax: set = warp / 8, 16 rows per warp, a row pair per quad of threads =================
    // (after a timed-out wait the threads keep going through the motions: later waits return at once)
    const int set = warp >> 3, w8 = warp & 7;
    const int qd = warp & 3, hf = (warp >> 2) & 1;
    const int q4 = lane & 3;
    const int rowA = qd * 32 + hf * 16 + (lane >> 2);  // my two rows of the tile: rowA and rowA + 8
    const uint32_t lane16 = (uint32_t)(qd * 32 + hf * 16) << 16;
    const uint32_t t_o = tmem + lane16 + TTM_O;
    float* mref_mine = mref + set * TBM + qd * 32 + hf * 16;
    const volatile float* mref_other = mref + (set ^ 1) * TBM + qd * 32 + hf * 16;
    const uint32_t bar_mx_mine = BAR(B_MX + 8 * set + w8), bar_mx_other = BAR(B_MX + 8 * (set ^ 1) + w8);
    // output share of the epilogue: 32 rows (thread = row) x 32 columns, the four warps of a quadrant side by side
    const int row = qd * 32 + lane, cq = set * 2 + hf;
    // tiles without any visible key (hand-made lists only): zeros
    for (int t = 0; t < ta; ++t) {
      const int t_row = q00 + t * TBM + row;
      if (t_row < s.Nq) {
        uint4* o4 = reinterpret_cast<uint4*>(out + (long long)h * s.os_h + (long long)t_row * s.os_t + cq * 32);
#pragma unroll
        for (int c = 0; c < 4; ++c) o4[c] = make_uint4(0, 0, 0, 0);
      }
    }
    int base_J = 0;  // number of the tile's first block in the CTA's stream
    for (int t = ta; t < tb; ++t) {
      const int nt = n_of(t), jm = tinfo[2 * t + 1];
      const int tq0 = q00 + t * TBM;
      tri::Rows st = {-INFINITY, -INFINITY, 0.f, 0.f};
      for (int j = (set ^ base_J) & 1; j < nt; j += 2) {
        const int J = base_J + j;
        const int b = J % 3;
        const bool masked = j >= jm;
        const int limA = masked ? rowA + tq0 + s.P - __ldg(indices + off + j) * BN - 2 * q4 : 0x7fffffff - 8;
        ok = tri::softmax_block<D, BN, SKIP>(tmem + lane16 + ttm_s(b), t_o, BAR(B_SFULL + b), (J / 3) & 1,
                                            BAR(B_ODONE + (J + 2) % 3), ((J - 1) / 3) & 1, BAR(B_PFULL + 2 * b), BAR(B_PFULL + 2 * b + 1), bar_mx_mine,
                                            bar_mx_other, ((J - 1) >> 1) & 1, mref_mine, mref_other, j == 0, masked, limA,
                                            scale_log2, skip_log2, lane, status, st) && ok;
      }
      // ---- the tile's epilogue ----
      const int J_last = base_J + nt - 1;
      if (((J_last ^ set) & 1) != 0) {
        // the other set had the last block: its final reference is the one my sums have to be brought to
        ok = mbar_wait(bar_mx_other, (J_last >> 1) & 1, status) && ok;
        ok = __all_sync(0xffffffffu, ok);
        const float pmA = mref_other[lane >> 2], pmB = mref_other[(lane >> 2) + 8];
        st.lA = tri::realign(st.lA, st.mrA, pmA, scale_log2);
        st.lB = tri::realign(st.lB, st.mrB, pmB, scale_log2);
      }
      st.lA += __shfl_xor_sync(0xffffffffu, st.lA, 1);
      st.lB += __shfl_xor_sync(0xffffffffu, st.lB, 1);
      st.lA += __shfl_xor_sync(0xffffffffu, st.lA, 2);
      st.lB += __shfl_xor_sync(0xffffffffu, st.lB, 2);
      float* ls = lsum + (t & 1) * 2 * TBM;
      if (q4 == 0) {
        ls[set * TBM + rowA] = st.lA;
        ls[set * TBM + rowA + 8] = st.lB;
      }
      asm volatile("bar.sync %0, %1;" ::"r"(1 + qd), "r"(128) : "memory");  // the four warps of this quadrant
      const float l_row = ls[row] + ls[TBM + row];
      ok = mbar_wait(BAR(B_ODONE + J_last % 3), (J_last / 3) & 1, status) && ok;
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      uint32_t o[32];
      tmem_ld32(tmem + ((uint32_t)(qd * 32) << 16) + TTM_O + cq * 32, o);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_OREAD));  // O has left tensor memory: the next tile's first P.V may overwrite it
      const int t_row = tq0 + row;
      if (ok && t_row < s.Nq) {  // rows beyond the sequence join the warp-wide loads, only their stores are dropped
        const float inv = l_row > 0.f ? 1.0f / l_row : 0.f;
        uint4* o4 = reinterpret_cast<uint4*>(out + (long long)h * s.os_h + (long long)t_row * s.os_t + cq * 32);
#pragma unroll
        for (int v4 = 0; v4 < 4; ++v4) {
          uint32_t wv[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            __nv_bfloat162 bb = __floats2bfloat162_rn(__uint_as_float(o[v4 * 8 + 2 * e]) * inv,
                                                      __uint_as_float(o[v4 * 8 + 2 * e + 1]) * inv);
            wv[e] = *reinterpret_cast<uint32_t*>(&bb);
          }
          o4[v4] = make_uint4(wv[0], wv[1], wv[2], wv[3]);
        }
      }
      base_J += nt;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 16) {
    tc_fence_after();
    tmem_dealloc(tmem, TTM_COLS);
  }
}

int launch_attention_tri(const Shape& s, const AttnArgs& a, cudaStream_t st) {
  constexpr int D = 128, BN = 128;
  using L = TriSmem<D, BN>;
  static_assert(L::DYN_BYTES <= 232448, "shared memory budget exceeded");
  if (!a.items) return EI_ERR_INVALID_ARG;
  CUtensorMap tmq, tmk, tmv;
  if (!make_tensor_map(&tmq, a.q, D, s.Nq, s.H, s.qs_t, s.qs_h, TBM) ||
      !make_tensor_map(&tmk, a.k, D, s.N, s.Hkv, s.ks_t, s.ks_h, BN) ||
      !make_tensor_map(&tmv, a.v, D, s.N, s.Hkv, s.vs_t, s.vs_h, BN))
    return EI_ERR_CUDA;
  const int tiles_per_seg = s.L_S / TBM;
  int NT = a.tri_tiles > 0 ? a.tri_tiles : 4;
  while (NT > 1 && (tiles_per_seg % NT != 0 || NT > TRI_MAXT)) NT >>= 1;
  const long long grid = (long long)s.H * s.C_S * (tiles_per_seg / NT);
  const float scale_log2 = a.scale * 1.4426950408889634f;
  const bool skip = a.skip_log2 < INFINITY;
  auto kern = skip ? sparse_attention_tri_kernel<D, BN, true> : sparse_attention_tri_kernel<D, BN, false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES) != cudaSuccess)
    return EI_ERR_CUDA;
  kern<<<(unsigned)grid, TRI_THREADS, L::DYN_BYTES, st>>>(tmq, tmk, tmv, a.out, a.items, a.indices, a.status, s, scale_log2,
                                                         a.skip_log2, NT);
  return cudaGetLastError() == cudaSuccess ? EI_OK : EI_ERR_CUDA;
}

}  // namespace ei
