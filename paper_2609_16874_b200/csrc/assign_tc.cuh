// Stage 4+5, Blackwell path: pixel-to-instance assignment (Eq. 4, Eq. 7, Eq. 8) with the pixels x D x K score
// contraction on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor memory) as a FILTER, and the
// decision taken exactly in binary32.
//
// For a pixel with halves xhat, yhat and a peak k with palette rows ex = P_w(a_k), ey = P_h(b_k):
//     A_k = ||xhat - ex||^2 = ||xhat||^2 + F - 2 xhat.ex,   B_k likewise,   d_k = sqrt(A_k) + sqrt(B_k).
// With S = A + B and Delta = A - B,
//     L := 2 S - |Delta| = max(A,B) + 3 min(A,B)   and   S <= L <= d^2 <= 2 S.
// S and Delta are each one dot product over all 4F channels away from a per-pixel constant (Delta takes the y half
// with the opposite sign, which the instruction descriptor's negate bit supplies).  The tensor cores deliver, for a
// tile of 128 pixels x 64 peaks, S_k and Delta_k into tensor memory, the accumulators having been pre-loaded with
// the per-pixel constants lowered by every error of the approximation (binary16 rounding of the palette and, for
// binary32 inputs, of the pixel; accumulation), and each thread, owning ONE pixel row, reads its row back with
// tcgen05.ld:
//   pass 1   the smallest S_k (the second smallest when the runner-up is wanted): d_best^2 <= 2 (S_min + slack) =: thr,
//            so a peak with L_k > thr cannot be the arg-min.                             1/2 instruction per pair
//   pass 2   L_k <= thr as a bit mask per row.                                           3 instructions per pair
//   A row with one bit is decided (no scores wanted, tau = +inf).  A row with several keeps them in registers and
//   its thread re-scores them in binary32 in the one fixed operation order that defines the result; a row with more
//   than kTcCand scores every peak.
//
// Work decomposition: a CTA walks spans of consecutive pixels; it compacts the span's participating 8-pixel groups
// and gathers 32 groups (256 rows) at a time with 16-byte asynchronous copies into a shared-memory tile that already
// is the MMA's A operand (pixel-major core matrices, no swizzle; the planar [channel][pixel] input needs no
// transpose).  The eight threads that fetch a group's channels also reduce the squared norms of its eight pixels
// among themselves, each ending up with the norms of the row it owns: one barrier per MMA round is all the
// synchronisation a tile needs.  The peak operand (K-major, rows -2 ex | -2 ey in binary16) is resident in shared
// memory.  One thread issues the MMAs of a round (2 row blocks x {S, Delta} x 4F/16 k-steps); everybody waits on an
// mbarrier with a bounded spin.  Two CTAs per SM, 256 tensor-memory columns each.
#pragma once

#include "assign_mma.cuh"
#include "cpe_common.cuh"

namespace cpe {

#ifdef CPE_TC_PROF
__device__ unsigned long long g_tc_prof[16];
#define TC_PROF(i) do { if (tid == 0) { const long long t_ = clock64(); atomicAdd(&g_tc_prof[i], (unsigned long long)(t_ - prof_t)); prof_t = t_; } } while (0)
#else
#define TC_PROF(i) do { } while (0)
#endif

constexpr int kTcThreads = 256;
constexpr int kTcRows = 256;        // rows (pixels) per tile: two MMA row blocks of 128
constexpr int kTcRound = 64;        // peaks per MMA round: S and Delta of both row blocks fill 256 tensor-memory columns
constexpr int kTcCols = 256;        // tensor-memory columns allocated per CTA
constexpr int kTcCand = 6;          // candidates a row keeps; more than that and it scores every peak
constexpr int kTcQueue = 3072;      // queue slots (8 bytes): per undecided row a header and one slot per candidate
constexpr int kTcFlushAt = kTcQueue - kTcRows * (kTcCand + 1);   // above this a tile's pushes might not fit: score first
constexpr int kTcHardQueue = 512;   // rows that score every peak
constexpr int kTcHardFlushAt = kTcHardQueue - kTcRows;
constexpr uint32_t kTcHeader = 0x80000000u;
constexpr int kTcWaitLimit = 1 << 20;

struct TcSmem {
  int tile, tile2, peaks, lab, queue, hardq, glist, gbits, misc, total;
};

// peak_cap must be a multiple of kTcRound
__host__ __device__ inline TcSmem tc_smem_layout(int KA, int peak_cap, int span, int two_tiles) {
  TcSmem s;
  int off = 0;
  s.tile = off;   off += 2 * KA * kTcRows * 2;
  s.tile2 = off;  off += two_tiles ? 2 * KA * kTcRows * 2 : 0;
  s.peaks = off;  off += peak_cap * 2 * KA * 2;
  s.lab = off;    off += span * 4;
  s.queue = off;  off += kTcQueue * 8;
  s.hardq = off;  off += kTcHardQueue * 4;
  s.glist = off;  off += 256 * 2;
  s.gbits = off;  off += 256;
  s.misc = off;   off += 128;   // scan scratch (9 ints), queue counters, tensor-memory base, mbarrier
  s.total = off;
  return s;
}

// ---- tcgen05 / mbarrier wrappers (PTX ISA: tcgen05 family, sm_100a)

// Shared-memory matrix descriptor, no swizzle: start address, "leading" byte offset = distance between core
// matrices along K, "stride" byte offset = distance between core matrices along M/N; a core matrix is 8 rows of 16 bytes.
__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3fffu);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
  d |= (uint64_t)1 << 46;
  return d;
}
// Instruction descriptor of kind::f16: binary32 accumulate (bit 4), binary16 A and B, A pixel-major (bit 15), B K-major,
// N/8 at bit 17, M/16 at bit 24; bit 14 negates B.
constexpr uint32_t kTcIdesc = (1u << 4) | (1u << 15) | ((uint32_t)(kTcRound >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
constexpr uint32_t kTcNegB = 1u << 14;

__device__ __forceinline__ void tc_mma(uint32_t taddr, uint64_t adesc, uint64_t bdesc, uint32_t idesc) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(taddr), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(1u)
      : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t mbar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mbar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Bounded wait for the given phase of an mbarrier; false if the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t mbar, uint32_t parity) {
  uint32_t done = 0;
  for (int it = 0; it < kTcWaitLimit && !done; ++it) {
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(done) : "r"(mbar), "r"(parity) : "memory");
  }
  return done != 0;
}

// 32 consecutive columns of this thread's tensor-memory lane from each of two addresses; the wait is part of the same
// statement so that no use of the values can be scheduled before it
__device__ __forceinline__ void tc_ld32x2(uint32_t ta, uint32_t tb, float (&va)[32], float (&vb)[32]) {
  uint32_t r[32], q[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%64];\n"
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63}, [%65];\n"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]),
        "=r"(q[0]), "=r"(q[1]), "=r"(q[2]), "=r"(q[3]), "=r"(q[4]), "=r"(q[5]), "=r"(q[6]), "=r"(q[7]), "=r"(q[8]),
        "=r"(q[9]), "=r"(q[10]), "=r"(q[11]), "=r"(q[12]), "=r"(q[13]), "=r"(q[14]), "=r"(q[15]), "=r"(q[16]),
        "=r"(q[17]), "=r"(q[18]), "=r"(q[19]), "=r"(q[20]), "=r"(q[21]), "=r"(q[22]), "=r"(q[23]), "=r"(q[24]),
        "=r"(q[25]), "=r"(q[26]), "=r"(q[27]), "=r"(q[28]), "=r"(q[29]), "=r"(q[30]), "=r"(q[31])
      : "r"(ta), "r"(tb)
      : "memory");
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    va[j] = __uint_as_float(r[j]);
    vb[j] = __uint_as_float(q[j]);
  }
}
__device__ __forceinline__ void tc_ld32(uint32_t ta, float (&va)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(ta)
      : "memory");
#pragma unroll
  for (int j = 0; j < 32; ++j) va[j] = __uint_as_float(r[j]);
}
// the same value into 32 consecutive columns of this thread's lane
__device__ __forceinline__ void tc_st32_fill(uint32_t taddr, float value) {
  const uint32_t c = __float_as_uint(value);
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};" ::"r"(taddr), "r"(c)
      : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float min3f(float a, float b, float c) {
  float r;
  asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// Offset, in halves, of element (row m, k-slot s) in a tile of kTcRows rows stored as pixel-major core matrices:
// a core matrix holds 8 k-slots x 8 rows, 16 bytes (8 rows) per k-slot; cores are contiguous along the rows.
__device__ __forceinline__ int tc_tile_off(int m, int s) { return (s >> 3) * (kTcRows * 8) + (m >> 3) * 64 + (s & 7) * 8 + (m & 7); }

// Sum over the 8 lanes of an aligned lane group of 8 values each, lane j of the group ending up with the total
// of value j (7 exchanges).
__device__ __forceinline__ float reduce_scatter8(const float (&a)[8], int j) {
  float b4[4], b2[2];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const float send = (j & 4) ? a[r] : a[r + 4], keep = (j & 4) ? a[r + 4] : a[r];
    b4[r] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const float send = (j & 2) ? b4[r] : b4[r + 2], keep = (j & 2) ? b4[r + 2] : b4[r];
    b2[r] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
  }
  const float send = (j & 1) ? b2[0] : b2[1], keep = (j & 1) ? b2[1] : b2[0];
  return keep + __shfl_xor_sync(0xffffffffu, send, 1);
}

// What the scoring step needs to know about the image and the CTA's shared memory.
template <typename T>
struct TcScore {
  const T* e_img;
  const float* pk_img;
  size_t plane;
  int F, K;
  float tau;
  int32_t* s_lab;
  int32_t* lab_img;
  float* best_img;
  float* second_img;
  unsigned long long* s_queue;
  uint32_t* s_hardq;
  uint32_t* s_qn;      // [0] queue slots in use, [1] hard rows listed
  uint32_t* status;
};

// The decision, in binary32, in the one fixed operation order that defines the result:
//   sx = 0; for c: t = xhat_c - ex_c; sx = fma(t, t, sx)  (likewise sy);  d = sqrt(sx) + sqrt(sy)
template <typename T, int KA>
__device__ __forceinline__ float tc_exact(const TcScore<T>& sc, uint32_t pix, int k) {
  const int F = sc.F;
  const T* src = sc.e_img + pix;
  const float* pk = sc.pk_img + (size_t)k * 4 * F;
  float s[2];
#pragma unroll
  for (int axis = 0; axis < 2; ++axis) {
    float acc = 0.0f;
#pragma unroll
    for (int cb = 0; cb < KA; cb += 16) {
      float pv[16], qv[16];   // the loads of 16 channels are issued before the chain consumes them
#pragma unroll
      for (int c = 0; c < 16; ++c)
        if (cb + c < 2 * F) {
          pv[c] = Elem<T>::load1(src + (size_t)(axis * 2 * F + cb + c) * sc.plane);
          qv[c] = __ldg(pk + axis * 2 * F + cb + c);
        }
#pragma unroll
      for (int c = 0; c < 16; ++c)
        if (cb + c < 2 * F) {
          const float v = __fsub_rn(pv[c], qv[c]);
          acc = __fmaf_rn(v, v, acc);
        }
    }
    s[axis] = acc;
  }
  return __fadd_rn(__fsqrt_rn(s[0]), __fsqrt_rn(s[1]));
}

// A pixel of the span whose labels are still staged in shared memory gets its label there; an earlier span's
// label map has been stored already, so the label goes to the map itself.
template <typename T>
__device__ __forceinline__ void tc_write_outcome(const TcScore<T>& sc, long long span0, int span_len, uint32_t pix, bool ok,
                                                 float d1, float d2, int k1, uint32_t& rejected) {
  const float inf = __int_as_float(0x7f800000);
  if (ok && k1 >= 0) {
    if (d1 < sc.tau) {
      const long long rel = (long long)pix - span0;
      if (rel >= 0 && rel < span_len) sc.s_lab[rel] = k1 + 1;
      else sc.lab_img[pix] = k1 + 1;
    } else {
      ++rejected;
    }
  }
  if (sc.best_img) {
    sc.best_img[pix] = ok ? d1 : inf;
    sc.second_img[pix] = ok ? d2 : inf;
  }
}

// Scores everything queued so far, all threads busy: one thread per (pixel, candidate) pair, then one thread per
// pixel picks the winner among its pairs; a warp per pixel that scores every peak.  Called by all threads of the CTA
// right after a barrier; nobody pushes while it runs.  A function of its own: one copy, its own registers.
template <typename T, int KA>
__device__ __noinline__ void tc_flush(const TcScore<T>& sc, long long span0, int span_len, uint32_t& rejected,
                                      uint32_t& n_full) {
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const float inf = __int_as_float(0x7f800000);
  const int n = (int)min(*reinterpret_cast<volatile uint32_t*>(sc.s_qn), (uint32_t)kTcQueue);
  const int nh = (int)min(*reinterpret_cast<volatile uint32_t*>(sc.s_qn + 1), (uint32_t)kTcHardQueue);
  const int K = sc.K, F = sc.F;
  unsigned long long* Q = sc.s_queue;
  // pairs: (pixel << 32 | k)  ->  (score << 32 | k)
  for (int e = tid; e < n; e += kTcThreads) {
    const unsigned long long v = Q[e];
    const uint32_t lo = (uint32_t)v, pix = (uint32_t)(v >> 32);
    if (lo & kTcHeader) continue;
    float d = inf;
    if (am_ok((int)lo < K, 5u, sc.status)) d = tc_exact<T, KA>(sc, pix, (int)lo);
    Q[e] = ((unsigned long long)__float_as_uint(d) << 32) | lo;
  }
  // rows that score every peak (pixels beyond the binary16 range, or too many candidates): a warp per row
  for (int h = wid; h < nh; h += kTcThreads / 32) {
    const uint32_t pix = sc.s_hardq[h];
    bool ok = true;
    if constexpr (sizeof(T) == 4) {
      // the binary16 copy could not tell an out-of-range value from a non-finite one: look at the originals
      const T* src = sc.e_img + pix;
      float fin = 0.0f;
      for (int l = lane; l < 2 * F; l += 32)
        fin = fold_finite(fin, Elem<T>::load1(src + (size_t)(2 * l) * sc.plane), Elem<T>::load1(src + (size_t)(2 * l + 1) * sc.plane));
      ok = !__any_sync(0xffffffffu, fin != fin);
    }
    float d1 = inf, d2 = inf;
    int k1 = -1;
    if (ok) {
#pragma unroll 1
      for (int k = lane; k < K; k += 32) {
        const float d = tc_exact<T, KA>(sc, pix, k);
        if (d < d1) { d2 = d1; d1 = d; k1 = k; }
        else if (d < d2) { d2 = d; }
      }
      unsigned long long bestp = pack_dk(d1, k1);
#pragma unroll
      for (int x = 16; x > 0; x >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xffffffffu, bestp, x);
        bestp = o < bestp ? o : bestp;
      }
      // the runner-up: every lane's best except the winner's, whose second counts instead
      float r2 = (k1 == pack_k(bestp)) ? d2 : d1;
#pragma unroll
      for (int x = 16; x > 0; x >>= 1) r2 = fminf(r2, __shfl_xor_sync(0xffffffffu, r2, x));
      d1 = pack_d(bestp);
      k1 = pack_k(bestp);
      d2 = r2;
    }
    if (lane == 0) {
      if (ok) ++n_full;
      tc_write_outcome(sc, span0, span_len, pix, ok, d1, d2, k1, rejected);
    }
  }
  __syncthreads();
  if (tid == 0) {
    sc.s_qn[0] = 0;      // everybody has read the counts; nobody pushes before this function's last barrier
    sc.s_qn[1] = 0;
  }
  // headers: (pixel << 32 | header bit | count); the row's pairs follow in ascending k, so that the lowest k keeps a tie
  for (int e = tid; e < n; e += kTcThreads) {
    const unsigned long long v = Q[e];
    const uint32_t lo = (uint32_t)v, pix = (uint32_t)(v >> 32);
    if (!(lo & kTcHeader)) continue;
    const int cnt = (int)(lo & 0xffu);
    if (!am_ok(cnt <= kTcCand && e + cnt < kTcQueue, 4u, sc.status)) continue;
    float d1 = inf, d2 = inf;
    int k1 = -1;
    for (int i = 1; i <= cnt; ++i) {
      const unsigned long long w = Q[e + i];
      const float d = __uint_as_float((uint32_t)(w >> 32));
      const int k = (int)(uint32_t)w;
      if (d < d1) { d2 = d1; d1 = d; k1 = k; }
      else if (d < d2) { d2 = d; }
    }
    tc_write_outcome(sc, span0, span_len, pix, true, d1, d2, k1, rejected);
  }
  __syncthreads();
}

// Requires 16-byte aligned planes: emb 16-byte aligned and HW a multiple of 8 (the caller falls back to the
// mma.sync kernel otherwise).  KA = 16 serves F <= 8, KA = 32 serves F <= 16.
template <typename T, int KA, bool WANT2>
__global__ void __launch_bounds__(kTcThreads, 2)
assign_tc_kernel(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int F, int K_max,
                 const float* __restrict__ peak_emb, const int32_t* __restrict__ count_ptr, float tau, int need_exact,
                 int peak_cap, int span, int vec_mask, int32_t* __restrict__ labels, float* __restrict__ best,
                 float* __restrict__ second, uint32_t* __restrict__ counters, uint32_t* __restrict__ status_all,
                 uint32_t* __restrict__ votes, int cells, int k_min) {
  constexpr int KS = KA / 16;                       // k-steps per axis
  constexpr int kTileHalves = 2 * KA * kTcRows;
  constexpr uint32_t kTileLbo = kTcRows * 16;       // bytes between core matrices along K in the tile
  extern __shared__ __align__(1024) unsigned char tc_smem[];
  constexpr int two_tiles = (sizeof(T) == 2 && KA == 16) ? 1 : 0;   // prefetch the next tile while this one is swept
  const TcSmem L = tc_smem_layout(KA, peak_cap, span, two_tiles);
  int32_t* s_lab = reinterpret_cast<int32_t*>(tc_smem + L.lab);
  __half* s_tile0 = reinterpret_cast<__half*>(tc_smem + L.tile);
  __half* s_pk = reinterpret_cast<__half*>(tc_smem + L.peaks);
  uint16_t* s_glist = reinterpret_cast<uint16_t*>(tc_smem + L.glist);     // participating 8-pixel groups of the span
  uint8_t* s_gbits = reinterpret_cast<uint8_t*>(tc_smem + L.gbits);       // which of a group's 8 pixels participate
  unsigned long long* s_queue = reinterpret_cast<unsigned long long*>(tc_smem + L.queue);
  uint32_t* s_hardq = reinterpret_cast<uint32_t*>(tc_smem + L.hardq);
  int* s_scan = reinterpret_cast<int*>(tc_smem + L.misc);                 // [0..8] warp offsets and total
  uint32_t* s_qn = reinterpret_cast<uint32_t*>(s_scan + 10);              // [0] queue slots in use, [1] hard rows listed
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_scan + 12);
  uint64_t* s_mbar = reinterpret_cast<uint64_t*>(tc_smem + L.misc + 64);

  const int b = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  uint32_t* status = status_all + b;
  // the vote map has no reader left: leave it zero for the next decode (votes == NULL keeps it)
  if (votes) zero_votes_share(votes + (size_t)b * cells, cells, (int)blockIdx.x, (int)gridDim.x);
  const size_t plane = (size_t)HW;
  const int D = 4 * F;
  const T* e_img = emb + (size_t)b * D * plane;
  const uint8_t* fg_img = fg ? fg + (size_t)b * plane : nullptr;
  const float* pk_img = peak_emb + (size_t)b * K_max * D;
  const int K = count_ptr[b];
  if (K < k_min) return;     // few peaks: this image is done by the plain all-pairs kernel launched next to this one
  const float inf = __int_as_float(0x7f800000);
  const float qnan = __int_as_float(0x7fc00000);
  const int n_spans = (HW + span - 1) / span;
  const int n_pchunks = K > 0 ? (K + peak_cap - 1) / peak_cap : 0;
  int32_t* lab_img = labels + (size_t)b * plane;
  float* best_img = best ? best + (size_t)b * plane : nullptr;
  float* second_img = second ? second + (size_t)b * plane : nullptr;
  const int n_grp_span = span >> 3;                 // 8-pixel groups per span (<= 256): thread t owns group t
  const uint32_t mbar = (uint32_t)__cvta_generic_to_shared(s_mbar);
  const uint32_t pk_lbo = (uint32_t)peak_cap * 16u; // bytes between core matrices along K in the peak operand
  const bool score_all = WANT2 || need_exact;       // scores wanted: every passing pair is re-scored
  const bool one_round = n_pchunks == 1 && K <= kTcRound;   // pass 2 finds pass 1's accumulators still in tensor memory
  // a row's 8 pixels = the 8 lanes gl*8 .. gl*8+7; lane cq fetches channels cq, cq+8, ... of group gl and owns row tid
  const int gl = tid >> 3, cq = tid & 7;

  // ---- one-time set-up: tensor memory, barrier, zeroed tiles (padding k-slots must stay zero), peak operand
  if (wid == 0) {
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(s_tmem);
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst), "r"(kTcCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(mbar) : "memory");
    s_qn[0] = 0;
    s_qn[1] = 0;
  }
  for (int i = tid; i < (1 + two_tiles) * kTileHalves / 2; i += kTcThreads) reinterpret_cast<uint32_t*>(s_tile0)[i] = 0u;

  // peak operand, K-major core matrices: row k = [-2 ex (2F), 0.., -2 ey (2F), 0..] in binary16 (the factor -2 is
  // exact); rows beyond the last peak are NaN, so that their columns never win a minimum nor pass a comparison
  auto load_peaks = [&](int pc) {
    const int k0 = pc * peak_cap;
    const int kn = min(peak_cap, K - k0);
    const int kn_r = (kn + kTcRound - 1) / kTcRound * kTcRound;
    for (int i = tid; i < kn_r * 2 * KA; i += kTcThreads) {
      const int k = i / (2 * KA), s = i - k * 2 * KA;
      const int axis = s / KA, cc = s - axis * KA;
      float v = 0.0f;
      if (k >= kn) v = qnan;
      else if (cc < 2 * F) v = -2.0f * pk_img[(size_t)(k0 + k) * D + axis * 2 * F + cc];
      s_pk[(s >> 3) * (peak_cap * 8) + k * 8 + (s & 7)] = __float2half_rn(v);
    }
    fence_async_smem();
  };
  if (n_pchunks == 1) load_peaks(0);
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  // this thread's row of the tile: row block mt = wid / 4 uses tensor-memory columns [128 mt, 128 mt + 128):
  // S in the first 64, Delta in the last 64; a warp reaches the 32 lanes 32 (wid % 4) ...
  const uint32_t t_row = tmem + ((uint32_t)((wid & 3) * 32) << 16) + (uint32_t)((wid >> 2) * 128);
  uint32_t phase = 0;
  bool failed = false, timed_out = false;

  // MMAs of one round: peaks [n0, n0 + 64) of the resident chunk against both row blocks of the tile
  auto issue_round = [&](const __half* tile, int n0, bool with_delta) {
    const uint32_t a0 = (uint32_t)__cvta_generic_to_shared(tile);
    const uint32_t b0 = (uint32_t)__cvta_generic_to_shared(s_pk) + (uint32_t)n0 * 16u;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int acc = 0; acc < 2; ++acc) {
        if (acc == 1 && !with_delta) continue;
#pragma unroll
        for (int ks = 0; ks < 2 * KS; ++ks) {
          const uint64_t da = tc_desc(a0 + (uint32_t)ks * 2u * kTileLbo + (uint32_t)mt * 2048u, kTileLbo, 128u);
          const uint64_t db = tc_desc(b0 + (uint32_t)ks * 2u * pk_lbo, pk_lbo, 128u);
          const uint32_t id = (acc == 1 && ks >= KS) ? (kTcIdesc | kTcNegB) : kTcIdesc;
          tc_mma(tmem + (uint32_t)(mt * 128 + acc * 64), da, db, id);
        }
      }
    tc_commit(mbar);
  };

  uint32_t rejected = 0, n_pairs = 0, n_rescored = 0, n_full = 0;
  TcScore<T> sc;
  sc.e_img = e_img; sc.pk_img = pk_img; sc.plane = plane; sc.F = F; sc.K = K; sc.tau = tau;
  sc.s_lab = s_lab; sc.lab_img = lab_img; sc.best_img = best_img; sc.second_img = second_img;
  sc.s_queue = s_queue; sc.s_hardq = s_hardq; sc.s_qn = s_qn; sc.status = status;
#ifdef CPE_TC_PROF
  long long prof_t = clock64();
#endif

  for (int sp = blockIdx.x; sp < n_spans && !failed; sp += gridDim.x) {
    // later spans first: the tail of the voting pass is what is still in L2
    const long long span0 = (long long)(n_spans - 1 - sp) * span;
    const int span_len = (int)min((long long)span, (long long)HW - span0);

    // ---- mask pass and compaction of the span's participating 8-pixel groups; background pixels get their outputs here
    {
      const long long p0 = span0 + (long long)tid * 8;
      const bool mine = tid < n_grp_span && p0 < HW;     // HW is a multiple of 8: the whole group is inside
      uint32_t bits = 0;
      if (mine) {
        if (!fg_img) {
          bits = 0xffu;
        } else if (vec_mask) {
          const uint2 w = __ldg(reinterpret_cast<const uint2*>(fg_img + p0));
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            bits |= (((w.x >> (8 * j)) & 0xffu) ? 1u : 0u) << j;
            bits |= (((w.y >> (8 * j)) & 0xffu) ? 1u : 0u) << (4 + j);
          }
        } else {
          for (int j = 0; j < 8; ++j)
            if (__ldg(fg_img + p0 + j)) bits |= 1u << j;
        }
        if (best_img) {
          for (int j = 0; j < 8; ++j)
            if (K == 0 || !((bits >> j) & 1u)) {
              best_img[p0 + j] = inf;
              second_img[p0 + j] = inf;
            }
        }
      }
      for (int i = tid; i < span / 4; i += kTcThreads) reinterpret_cast<int4*>(s_lab)[i] = make_int4(0, 0, 0, 0);
      const uint32_t gm = __ballot_sync(0xffffffffu, bits != 0);
      if (lane == 0) s_scan[wid] = __popc(gm);
      __syncthreads();
      if (tid == 0) {
        int run = 0;
#pragma unroll
        for (int w = 0; w < kTcThreads / 32; ++w) {
          const int v = s_scan[w];
          s_scan[w] = run;
          run += v;
        }
        s_scan[kTcThreads / 32] = run;
      }
      __syncthreads();
      if (bits) {
        const int gi = s_scan[wid] + __popc(gm & ((1u << lane) - 1u));
        s_glist[gi] = (uint16_t)tid;
        s_gbits[gi] = (uint8_t)bits;
      }
      __syncthreads();
    }
    const int n_groups = s_scan[kTcThreads / 32];
    const int n_chunks = K > 0 ? (n_groups + 31) / 32 : 0;
    TC_PROF(0);

    // One tile = 32 groups x 4F channels, 16 bytes (8 pixels of one channel) per copy, written where the MMA reads
    // them: k-slot s of group gl at core matrix (gl, s / 8), row s % 8.  This thread: group gl, channels cq, cq+8, ...
    auto slot_of = [&](int c) { return c >= 2 * F ? KA + (c - 2 * F) : c; };
    auto unit_ptr = [&](__half* tile, int c) {
      const int s = slot_of(c);
      return tile + (s >> 3) * (kTcRows * 8) + gl * 64 + (s & 7) * 8;
    };
    auto issue_gather = [&](int ci, __half* dst_tile) {
      if constexpr (sizeof(T) == 2) {
        const int gi = ci * 32 + gl;
        if (gi < n_groups) {
          const T* src0 = e_img + span0 + (int)s_glist[gi] * 8;
          for (int c = cq; c < D; c += 8) {
            const uint32_t d32 = (uint32_t)__cvta_generic_to_shared(unit_ptr(dst_tile, c));
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(d32), "l"(src0 + (size_t)c * plane));
          }
        }
        asm volatile("cp.async.commit_group;\n" ::);
      }
    };
    if (two_tiles && n_chunks > 0) issue_gather(0, s_tile0);

    for (int ci = 0; ci < n_chunks && !failed; ++ci) {
      __half* s_tile = two_tiles ? s_tile0 + (size_t)(ci & 1) * kTileHalves : s_tile0;
      const int gi = ci * 32 + gl;
      // ---- gather (or its completion) and the squared norms of the group's 8 pixels over this thread's channels
      float ax[8], ay[8];
#pragma unroll
      for (int r = 0; r < 8; ++r) ax[r] = ay[r] = 0.0f;
      auto add_squares = [&](const uint4& q, int c) {
        const __half2* h = reinterpret_cast<const __half2*>(&q);
        float t[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __half22float2(h[i]);
          t[2 * i] = f.x * f.x;
          t[2 * i + 1] = f.y * f.y;
        }
        if (c < 2 * F) {
#pragma unroll
          for (int r = 0; r < 8; ++r) ax[r] += t[r];
        } else {
#pragma unroll
          for (int r = 0; r < 8; ++r) ay[r] += t[r];
        }
      };
      if constexpr (sizeof(T) == 2) {
        if (!two_tiles) issue_gather(ci, s_tile);
        asm volatile("cp.async.wait_group 0;\n" ::: "memory");
        if (gi < n_groups)
          for (int c = cq; c < D; c += 8) add_squares(*reinterpret_cast<const uint4*>(unit_ptr(s_tile, c)), c);
      } else {
        // binary32: two 128-bit loads per unit, rounded to binary16 on the way
        if (gi < n_groups) {
          const T* src0 = e_img + span0 + (int)s_glist[gi] * 8;
          for (int c = cq; c < D; c += 8) {
            const float4* src = reinterpret_cast<const float4*>(src0 + (size_t)c * plane);
            const float4 lo = __ldg(src), hi = __ldg(src + 1);
            __half2 h[4] = {__floats2half2_rn(lo.x, lo.y), __floats2half2_rn(lo.z, lo.w),
                            __floats2half2_rn(hi.x, hi.y), __floats2half2_rn(hi.z, hi.w)};
            const uint4 q = *reinterpret_cast<const uint4*>(h);
            *reinterpret_cast<uint4*>(unit_ptr(s_tile, c)) = q;
            add_squares(q, c);
          }
        }
      }
      fence_async_smem();
      const float nx = reduce_scatter8(ax, cq), ny = reduce_scatter8(ay, cq);
      TC_PROF(1);

      // ---- this thread's row (pixel cq of group gl): error bounds, accumulator constants
      int off = 0xffff;
      if (gi < n_groups && ((s_gbits[gi] >> cq) & 1u)) off = (int)s_glist[gi] * 8 + cq;
      const bool present = off != 0xffff && am_ok(off < span_len, 1u, status);
      const bool finite = (nx + ny) < inf;
      // binary16 pixels: a non-finite norm is a non-finite pixel.  binary32 pixels: it may also be a value beyond
      // the binary16 range, so the row is scored exactly (and its finiteness checked there).
      bool valid = present && (finite || sizeof(T) == 4);
      bool hard = present && !finite && sizeof(T) == 4;
      const bool live = present && finite;
      float cS, cD, dS;      // accumulator constants; S_lo <= S <= S_lo + 2 dS and |Delta - Delta_c| <= dS
      {
        const float kappa = (sizeof(T) == 4 ? 3.0f : 1.0f) * 4.93e-4f;   // 2^-11 * 1.01 (x3: pixel rounding too)
        const float sq2f = sqrtf(2.0f * (float)F);
        const float nnx = live ? nx : 0.0f, nny = live ? ny : 0.0f;
        const float n1x = sq2f * sqrtf(nnx) * 1.0001f, n1y = sq2f * sqrtf(nny) * 1.0001f;   // sum |v| <= sqrt(2F) ||v||
        const float cfx = nnx + (float)F, cfy = nny + (float)F;
        // per axis: | true A - (||xhat||^2 + F + dot) | <= delta
        const float dx = kappa * n1x + 1e-5f * (cfx + 2.0f * n1x + 2.0f);
        const float dy = kappa * n1y + 1e-5f * (cfy + 2.0f * n1y + 2.0f);
        dS = (dx + dy) + 2e-6f * (cfx + cfy + 2.0f * (n1x + n1y) + 2.0f);   // plus the roundings of the constants
        cS = (cfx + cfy) - dS;
        cD = nnx - nny;
      }
      TC_PROF(2);

      // One round: constants into tensor memory, barrier, MMAs, wait.  Returns false, for every thread, once any
      // thread's wait has run out (the barrier itself carries the flag).
      bool first_round = true;
      auto run_round = [&](int n0, bool with_delta) -> bool {
        tc_st32_fill(t_row, cS);
        tc_st32_fill(t_row + 32, cS);
        if (with_delta) {
          tc_st32_fill(t_row + 64, cD);
          tc_st32_fill(t_row + 96, cD);
        }
        tc_wait_st();
        tc_fence_before();
        // the barrier also tells whether any wait has run out, and whether the queues have to be worked off before
        // this tile pushes (the last thread to arrive sees every push of the previous tile)
        const bool full = *reinterpret_cast<volatile uint32_t*>(s_qn) > (uint32_t)kTcFlushAt ||
                          *reinterpret_cast<volatile uint32_t*>(s_qn + 1) > (uint32_t)kTcHardFlushAt;
        bool flush = false;
        if (__syncthreads_or((timed_out || full) ? 1 : 0)) {
          if (__syncthreads_or(timed_out ? 1 : 0)) return false;
          flush = true;
        }
        if (tid == 0) {
          tc_fence_after();
          issue_round(s_tile, n0, with_delta);
        }
        // every thread is past the previous tile: its buffer can take the tile after this one
        if (first_round && two_tiles && ci + 1 < n_chunks) issue_gather(ci + 1, s_tile0 + (size_t)((ci + 1) & 1) * kTileHalves);
        first_round = false;
        if (flush) tc_flush<T, KA>(sc, span0, span_len, rejected, n_full);   // while the tensor cores work
        if (!mbar_wait(mbar, phase)) {
          timed_out = true;
          am_ok(false, 8u, status);
        }
        phase ^= 1u;
        tc_fence_after();
        return true;
      };

      // ---- pass 1: the smallest (and, if the runner-up is wanted, second smallest) S_k of the row
      float s1 = inf, s2 = inf;
      for (int pc = 0; pc < n_pchunks && !failed; ++pc) {
        if (n_pchunks > 1) { __syncthreads(); load_peaks(pc); __syncthreads(); }
        const int kn = min(peak_cap, K - pc * peak_cap);
        for (int n0 = 0; n0 < kn && !failed; n0 += kTcRound) {
          if (!run_round(n0, one_round)) { failed = true; break; }
          for (int c0 = 0; c0 < kTcRound && n0 + c0 < kn; c0 += 32) {
            float vS[32];
            tc_ld32(t_row + c0, vS);
            if constexpr (WANT2) {
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const float v = (vS[j] == vS[j]) ? vS[j] : inf;   // columns beyond the last peak are NaN
                const float lo = fminf(s1, v), hi = fmaxf(s1, v);
                s1 = lo;
                s2 = fminf(s2, hi);
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; j += 2) s1 = min3f(s1, vS[j], vS[j + 1]);
            }
          }
        }
      }
      if (failed) break;
      TC_PROF(3);
      // d_best^2 <= 2 S_true(arg-min) <= 2 (S_lo + 2 dS).  A peak can only win if L_true <= d_best^2, and what pass 2
      // computes, 2 S_lo - |Delta_c|, is at most L_true + dS: the test is 2 S_lo - |Delta_c| <= 2 (S_min + 2 dS) + dS.
      // Rows without a usable pixel get a NaN threshold: no comparison with it is ever true.
      const float sref = WANT2 ? s2 : s1;
      const float thr = live ? (2.0f * (sref + 2.0f * dS) * (1.0f + 1e-5f) + 1e-6f) + dS : qnan;

      // ---- pass 2: L_k <= thr as a bit mask; the peaks that pass are the row's candidates
      int cnt = 0, ck0 = -1, ck1 = -1, ck2 = -1, ck3 = -1, ck4 = -1, ck5 = -1;
      for (int pc = 0; pc < n_pchunks && !failed; ++pc) {
        if (n_pchunks > 1) { __syncthreads(); load_peaks(pc); __syncthreads(); }
        const int k0 = pc * peak_cap;
        const int kn = min(peak_cap, K - k0);
        for (int n0 = 0; n0 < kn && !failed; n0 += kTcRound) {
          if (!one_round && !run_round(n0, true)) { failed = true; break; }
          for (int c0 = 0; c0 < kTcRound && n0 + c0 < kn; c0 += 32) {
            float vS[32], vD[32];
            tc_ld32x2(t_row + c0, t_row + 64 + c0, vS, vD);
            uint32_t mk = 0;
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (fmaf(2.0f, vS[j], -fabsf(vD[j])) <= thr) mk |= 1u << j;
            const int rem = kn - (n0 + c0);
            if (rem < 32) mk &= (1u << rem) - 1u;
            if (mk) {
              const int kbase = k0 + n0 + c0;
              n_pairs += (uint32_t)__popc(mk);
              while (mk) {
                const int k = kbase + __ffs(mk) - 1;
                mk &= mk - 1;
                if (cnt == 0) ck0 = k;
                else if (cnt == 1) ck1 = k;
                else if (cnt == 2) ck2 = k;
                else if (cnt == 3) ck3 = k;
                else if (cnt == 4) ck4 = k;
                else if (cnt == 5) ck5 = k;
                ++cnt;
              }
            }
          }
        }
      }
      if (failed) break;
      if (live) am_ok(cnt > 0, 9u, status);                 // the arg-min always passes
      TC_PROF(4);

      // ---- the row's outcome: decided here, or queued for the scoring step
      if (valid && cnt > kTcCand) hard = true;
      if (present) {
        const uint32_t pix = (uint32_t)(span0 + off);
        int want_score = 0;                                 // (kept as separate statements)
        if (live && score_all) want_score = 1;
        if (live && cnt > 1) want_score = 1;
        if (hard) {
          const uint32_t hp = atomicAdd(s_qn + 1, 1u);
          if (am_ok(hp < (uint32_t)kTcHardQueue, 2u, status)) s_hardq[hp] = pix;
        } else if (want_score) {
          const uint32_t pos = atomicAdd(s_qn, (uint32_t)(1 + cnt));
          if (am_ok(pos + (uint32_t)cnt < (uint32_t)kTcQueue, 3u, status)) {
            const unsigned long long hi = (unsigned long long)pix << 32;
            s_queue[pos] = hi | kTcHeader | (uint32_t)cnt;
            s_queue[pos + 1] = hi | (uint32_t)ck0;
            if (cnt > 1) s_queue[pos + 2] = hi | (uint32_t)ck1;
            if (cnt > 2) s_queue[pos + 3] = hi | (uint32_t)ck2;
            if (cnt > 3) s_queue[pos + 4] = hi | (uint32_t)ck3;
            if (cnt > 4) s_queue[pos + 5] = hi | (uint32_t)ck4;
            if (cnt > 5) s_queue[pos + 6] = hi | (uint32_t)ck5;
            if (cnt > 1) ++n_rescored;
          }
        } else if (valid && cnt == 1) {
          s_lab[off] = ck0 + 1;                            // decided by the filter alone (tau = +inf, no scores)
        } else if (best_img) {
          best_img[pix] = inf;                             // a pixel that takes no part (non-finite)
          second_img[pix] = inf;
        }
      }
      TC_PROF(5);
    }
    if (failed) break;
    __syncthreads();
    TC_PROF(6);
    // ---- label map of the span: every pixel written, 128-bit stores when the span is aligned
    if ((span_len & 3) == 0 && ((uintptr_t)(lab_img + span0) & 15u) == 0) {
      for (int i = tid; i < span_len / 4; i += kTcThreads)
        reinterpret_cast<int4*>(lab_img + span0)[i] = reinterpret_cast<const int4*>(s_lab)[i];
    } else {
      for (int i = tid; i < span_len; i += kTcThreads) lab_img[span0 + i] = s_lab[i];
    }
    __syncthreads();
    TC_PROF(7);
  }

  // ---- what is still queued (every span's label map has been stored)
  __syncthreads();
  if (!failed) tc_flush<T, KA>(sc, -1, 0, rejected, n_full);

  // ---- tear-down: no copy in flight, tensor memory returned
  asm volatile("cp.async.wait_all;\n" ::: "memory");
  tc_fence_before();
  __syncthreads();
  if (wid == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTcCols) : "memory");

  const uint32_t wr = __reduce_add_sync(0xffffffffu, rejected);
  const uint32_t wp = __reduce_add_sync(0xffffffffu, n_pairs);
  const uint32_t ws = __reduce_add_sync(0xffffffffu, n_rescored);
  const uint32_t wf = __reduce_add_sync(0xffffffffu, n_full);
  if (lane == 0) {
    if (wr) atomicAdd(&counters[b * CPE_CNT_N + CPE_CNT_TAU_REJECTED], wr);
    if (wp) atomicAdd(&counters[b * CPE_CNT_N + CPE_CNT_FILTER_PAIRS], wp);
    if (ws) atomicAdd(&counters[b * CPE_CNT_N + CPE_CNT_RESCORED], ws);
    if (wf) atomicAdd(&counters[b * CPE_CNT_N + CPE_CNT_FULL_SCORED], wf);
  }
}

}  // namespace cpe
