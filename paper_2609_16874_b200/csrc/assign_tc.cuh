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
// tile of 128 pixels x 64 peaks, the two dot products into tensor memory; a thread that owns ONE pixel row reads
// the row back with tcgen05.ld and adds the row's constants, lowered by every error of the approximation
// (binary16 rounding of the palette and, for binary32 inputs, of the pixel; accumulation):
//   pass 1   the smallest S_k (the second smallest when the runner-up is wanted): d_best^2 <= 2 (S_min + slack) =: thr,
//            so a peak with L_k > thr cannot be the arg-min.                             1/2 instruction per pair
//            The minimum of every block of 32 columns is kept as well: |Delta| <= S bounds what pass 2 computes from
//            below by S alone, so a block whose minimum is too large for every row of the warp is skipped there.
//   pass 2   L_k <= thr as a bit mask per row, 4 instructions per pair.  A peak that passes gets bounds
//            dlo <= d_k <= dhi from its S and Delta; the smallest dhi bounds the best distance, and the row's
//            candidates are the peaks with dlo below it.  (The sweep runs as four chains, one per column number
//            mod 4, each remembering the values of its last passing column: registers cannot be indexed by a
//            run-time column number, and this way several passing columns of a block still have theirs at hand.)
//   A row with one candidate is decided (no scores wanted, tau = +inf).  The others are queued, per warp, and
//   worked off when the queue fills up, and at the end by all warps: one lane per (pixel, candidate) pair scores it
//   in binary32 in the one fixed operation order that defines the result, then one lane per pixel picks the winner.
//   A row with more than kTcCand candidates scores every peak, a warp per row.
//
// The CTA is a pipeline of two roles that meet only at mbarriers:
//   producers (4 warps)   take spans of 1024 pixels from a ticket counter: mask pass, compaction of the participating
//                         8-pixel groups into a ring; per tile of 16 groups (128 rows): 16-byte asynchronous copies
//                         straight into the MMA's A operand layout (pixel-major core matrices, no swizzle; the planar
//                         [channel][pixel] input needs no transpose), two tiles ahead; the 8 lanes that fetch a
//                         group's channels reduce the squared norms of its 8 pixels among themselves, each ending up
//                         with the norms of the row it describes; row data (pixel index, constants, slack, flags)
//                         into shared memory.  They never touch tensor memory.
//   consumers (4 warps)   wait for a stage, read their rows, release the stage, decide or queue, write labels (8 lanes
//                         = the 8 pixels of a group: full 32-byte sectors).  The last warp to release a stage issues
//                         the MMAs of the round after next into it (one lane: {S, Delta} x 4F/16 k-steps of M=128,
//                         N=64, committed to the stage's mbarrier and, with the tile's last round, to the tile
//                         buffer's).
// Two tensor-memory stages of 128 columns, four tile buffers (two for F > 8); two CTAs per SM.  Up to 64 peaks a
// tile takes one stage while the other one is filled for the next tile; 65 to 128 peaks take both stages for one tile
// (one round over all peaks: the MMAs of the next tile then wait for the release, the SM's other CTA fills the gap);
// more peaks than that go round by round, pass 1 over all rounds and then pass 2 (slower than the mma.sync kernel,
// which the launcher therefore prefers there).  Every wait is
// bounded; a wait that runs out raises a flag that every other wait polls, the status word records it, and the
// kernel winds down.  (A CTA of a kernel that uses tensor memory keeps the SM to itself until it has given up its
// right to allocate: hence the relinquish right after the allocation.)
#pragma once

#include "assign_mma.cuh"
#include "cpe_common.cuh"

namespace cpe {

constexpr int kTcThreads = 256;       // warps 0-3 consume (and issue the MMAs), warps 4-7 produce
constexpr int kTcRows = 128;          // rows (pixels) per tile: one MMA row block
constexpr int kTcGroups = kTcRows / 8;
constexpr int kTcRound = 64;          // peaks per MMA round: S and Delta fill one 128-column stage
constexpr int kTcCols = 256;          // tensor-memory columns allocated per CTA: two stages
constexpr int kTcMaxTiles = 4;        // tile buffers: 4 for F <= 8 (copies run two tiles ahead), 2 above (none ahead)
constexpr int kTcSpan = 1024;         // pixels per producer step: one 8-pixel group per producer thread
constexpr int kTcRing = 512;          // group ring entries (a span adds at most 128, a tile takes 16)
constexpr int kTcCand = 8;            // candidates a row keeps (in shared memory); more than that and it scores every peak
constexpr int kTcQueue = 768;         // queue slots (8 bytes) per consumer warp: a header and one slot per candidate
constexpr int kTcFlushAt = kTcQueue - 32 * (kTcCand + 1);   // above this a tile's pushes might not fit: score first
constexpr int kTcHardQueue = 64;      // rows that score every peak, per consumer warp
constexpr int kTcHardFlushAt = kTcHardQueue - 32;
constexpr uint32_t kTcHeader = 0x80000000u;
constexpr int kTcWaitLimit = 1 << 22;

// row flags handed from the producers to the consumers
constexpr uint32_t kRfGroup = 1u;     // the row belongs to a real group of the tile (its label is written)
constexpr uint32_t kRfPresent = 2u;   // ... and holds a participating pixel
constexpr uint32_t kRfLive = 4u;      // ... that is finite: the filter applies
constexpr uint32_t kRfHard = 8u;      // binary32 pixel beyond the binary16 range: score every peak
constexpr uint32_t kRfEnd = 16u;      // no more tiles

struct TcSmem {
  int tiles, peaks, queue, hardq, cand, clo, bmin, ring, ringbits, rpix, rslack, rcs, rcd, rflags, misc, total;
};

// peak_cap must be a multiple of kTcRound
__host__ __device__ constexpr int tc_tiles(int KA) { return KA == 16 ? 4 : 2; }

__host__ __device__ inline TcSmem tc_smem_layout(int KA, int peak_cap) {
  TcSmem s;
  int off = 0;
  s.tiles = off;    off += tc_tiles(KA) * 2 * KA * kTcRows * 2;
  s.peaks = off;    off += peak_cap * 2 * KA * 2;
  s.queue = off;    off += 4 * kTcQueue * 8;
  s.hardq = off;    off += 4 * kTcHardQueue * 4;
  s.cand = off;     off += kTcCand * kTcRows * 2;
  s.clo = off;      off += kTcCand * kTcRows * 4;
  s.bmin = off;     off += 4 * kTcRows * 4;
  s.ring = off;     off += kTcRing * 4;
  s.ringbits = off; off += kTcRing;
  s.rpix = off;     off += tc_tiles(KA) * kTcRows * 4;
  s.rslack = off;   off += tc_tiles(KA) * kTcRows * 4;
  s.rcs = off;      off += tc_tiles(KA) * kTcRows * 4;
  s.rcd = off;      off += tc_tiles(KA) * kTcRows * 4;
  s.rflags = off;   off += tc_tiles(KA) * kTcRows * 4;
  s.misc = off;     off += 256;   // producer scan scratch, abort flag, tensor-memory base, mbarriers
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

// D (tensor memory) = A B (+ D if accumulate)
__device__ __forceinline__ void tc_mma(uint32_t taddr, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(taddr), "l"(adesc), "l"(bdesc), "r"(idesc),
      "r"(accumulate ? 1u : 0u)
      : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t mbar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mbar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void mbar_init(uint32_t mbar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t mbar) {
  asm volatile("{\n.reg .b64 st;\nmbarrier.arrive.shared::cta.b64 st, [%0];\n}\n" ::"r"(mbar) : "memory");
}
// A bounded wait ran out: reported in the image's status word; the caller winds its CTA down (abort flag) and returns.
__device__ __forceinline__ void tc_timed_out(uint32_t* status) { atomicOr(status, (uint32_t)CPE_STATUS_TIMEOUT); }

// Bounded wait for the phase of the given parity; gives up early once the CTA's abort flag is up.  False: gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t mbar, uint32_t parity, const volatile int* abort_flag) {
  for (int it = 0; it < kTcWaitLimit; ++it) {
    uint32_t done;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(done) : "r"(mbar), "r"(parity) : "memory");
    if (done) return true;
    if ((it & 15) == 15 && *abort_flag) return false;
  }
  return false;
}
// Barrier among the 128 producer threads that also ORs a flag (barrier resource 1)
__device__ __forceinline__ bool producers_sync_or(bool flag) {
  uint32_t r;
  asm volatile(
      "{\n.reg .pred p, q;\nsetp.ne.b32 p, %1, 0;\nbarrier.cta.red.or.pred q, 1, 128, p;\nselp.u32 %0, 1, 0, q;\n}\n"
      : "=r"(r) : "r"(flag ? 1u : 0u) : "memory");
  return r != 0;
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
__device__ __forceinline__ float min3f(float a, float b, float c) {
  float r;
  asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

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

// What the scoring step needs to know about the image.
template <typename T>
struct TcScore {
  const T* e_img;
  const float* pk_img;
  size_t plane;
  int F, K;
  float tau;
  int32_t* lab_img;
  float* best_img;
  float* second_img;
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

template <typename T>
__device__ __forceinline__ void tc_write_outcome(const TcScore<T>& sc, uint32_t pix, bool ok, float d1, float d2, int k1,
                                                 uint32_t& rejected) {
  const float inf = __int_as_float(0x7f800000);
  int label = 0;
  if (ok && k1 >= 0) {
    if (d1 < sc.tau) label = k1 + 1; else ++rejected;
  }
  sc.lab_img[pix] = label;
  if (sc.best_img) {
    sc.best_img[pix] = ok ? d1 : inf;
    sc.second_img[pix] = ok ? d2 : inf;
  }
}

// Works off one consumer warp's queues, all lanes busy: one lane per (pixel, candidate) pair, then one lane per
// pixel picks the winner among its pairs; the whole warp for a pixel that scores every peak.  Called by all 32
// lanes of a warp; with n_parts > 1 several warps share the queue (part = which share) and the steps are separated
// by CTA barriers, so every thread of the CTA has to make the call (n = nh = 0 for a warp without a share).
// A function of its own: one copy, its own registers.
template <typename T, int KA>
__device__ __noinline__ void tc_flush_warp(const TcScore<T>& sc, unsigned long long* Q, int n, const uint32_t* H, int nh,
                                           int part, int n_parts, uint32_t& rejected, uint32_t& n_full) {
  const int lane = (threadIdx.x & 31) + 32 * part, stride = 32 * n_parts;
  const float inf = __int_as_float(0x7f800000);
  const int K = sc.K, F = sc.F;
  if (n_parts > 1) __syncthreads(); else __syncwarp();
  // pairs: (pixel << 32 | k)  ->  (score << 32 | k)
  for (int e = lane; e < n; e += stride) {
    const unsigned long long v = Q[e];
    const uint32_t lo = (uint32_t)v, pix = (uint32_t)(v >> 32);
    if (lo & kTcHeader) continue;
    float d = inf;
    if (am_ok((int)lo < K, 5u, sc.status)) d = tc_exact<T, KA>(sc, pix, (int)lo);
    Q[e] = ((unsigned long long)__float_as_uint(d) << 32) | lo;
  }
  if (n_parts > 1) __syncthreads(); else __syncwarp();
  // headers: (pixel << 32 | header bit | count); the row's pairs follow in ascending k, so that the lowest k keeps a tie
  for (int e = lane; e < n; e += stride) {
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
    tc_write_outcome(sc, pix, true, d1, d2, k1, rejected);
  }
  // rows that score every peak (pixels beyond the binary16 range, or too many candidates)
  const int wl = threadIdx.x & 31;   // lane within the warp
  for (int h = part; h < nh; h += n_parts) {
    const uint32_t pix = H[h];
    bool ok = true;
    if constexpr (sizeof(T) == 4) {
      // the binary16 copy could not tell an out-of-range value from a non-finite one: look at the originals
      const T* src = sc.e_img + pix;
      float fin = 0.0f;
      for (int l = wl; l < 2 * F; l += 32)
        fin = fold_finite(fin, Elem<T>::load1(src + (size_t)(2 * l) * sc.plane), Elem<T>::load1(src + (size_t)(2 * l + 1) * sc.plane));
      ok = !__any_sync(0xffffffffu, fin != fin);
    }
    float d1 = inf, d2 = inf;
    int k1 = -1;
    if (ok) {
#pragma unroll 1
      for (int k = wl; k < K; k += 32) {
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
    if (wl == 0) {
      if (ok) ++n_full;
      tc_write_outcome(sc, pix, ok, d1, d2, k1, rejected);
    }
  }
  __syncwarp();
}

// Requires 16-byte aligned planes: emb 16-byte aligned and HW a multiple of 8 (the caller takes the mma.sync kernel
// otherwise).  KA = 16 serves F <= 8, KA = 32 serves F <= 16.  Images with fewer than k_min or more than
// min(k_max, peak_cap) peaks are not touched.
template <typename T, int KA, bool WANT2>
__device__ __forceinline__ void
assign_tc_body(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int F, int K_max,
                 const float* __restrict__ peak_emb, const int32_t* __restrict__ count_ptr, float tau, int need_exact,
                 int peak_cap, int vec_mask, int32_t* __restrict__ labels, float* __restrict__ best,
                 float* __restrict__ second, uint32_t* __restrict__ counters, uint32_t* __restrict__ status_all,
                 uint32_t* __restrict__ votes, int cells, int k_min, int k_max, uint32_t* __restrict__ acc, int test_stall) {
  constexpr int KS = KA / 16;                       // k-steps per axis
  constexpr int kTiles = tc_tiles(KA);              // tile buffers
  constexpr int kAhead = kTiles - 2;                // tiles whose copies are in flight while one is being completed
  constexpr int kTileHalves = 2 * KA * kTcRows;
  constexpr uint32_t kTileLbo = kTcRows * 16;       // bytes between core matrices along K in a tile
  extern __shared__ __align__(1024) unsigned char tc_smem[];
  const TcSmem L = tc_smem_layout(KA, peak_cap);
  __half* s_tiles = reinterpret_cast<__half*>(tc_smem + L.tiles);
  __half* s_pk = reinterpret_cast<__half*>(tc_smem + L.peaks);
  unsigned long long* s_queue = reinterpret_cast<unsigned long long*>(tc_smem + L.queue);
  uint32_t* s_hardq = reinterpret_cast<uint32_t*>(tc_smem + L.hardq);
  uint16_t* s_cand = reinterpret_cast<uint16_t*>(tc_smem + L.cand);       // [slot][row]: the peaks that passed, per row
  float* s_clo = reinterpret_cast<float*>(tc_smem + L.clo);               // [slot][row]: their lower bounds of the distance
  float* s_bmin = reinterpret_cast<float*>(tc_smem + L.bmin);             // [block of 32 columns][row]: smallest S of pass 1
  uint32_t* s_ring = reinterpret_cast<uint32_t*>(tc_smem + L.ring);       // participating 8-pixel groups, in pixel order
  uint8_t* s_ringbits = reinterpret_cast<uint8_t*>(tc_smem + L.ringbits); // which of a group's 8 pixels participate
  uint32_t* s_rpix = reinterpret_cast<uint32_t*>(tc_smem + L.rpix);       // per tile buffer and row: pixel index
  float* s_rslack = reinterpret_cast<float*>(tc_smem + L.rslack);         // ... the row's error bound dS
  float* s_rcs = reinterpret_cast<float*>(tc_smem + L.rcs);               // ... S_lo = cS + the S accumulator
  float* s_rcd = reinterpret_cast<float*>(tc_smem + L.rcd);               // ... Delta = cD + the Delta accumulator
  uint32_t* s_rflags = reinterpret_cast<uint32_t*>(tc_smem + L.rflags);   // ... kRf* flags
  int* s_scan = reinterpret_cast<int*>(tc_smem + L.misc);                 // [0..3] producer warps' group counts
  volatile int* s_abort = s_scan + 8;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_scan + 9);
  int* s_qfill = s_scan + 10;                                             // [0..7] the consumer warps' queue fills at the end
  uint32_t* s_relcnt = reinterpret_cast<uint32_t*>(s_scan + 18);          // [2] releases of a stage so far
  volatile uint32_t* s_endtile = reinterpret_cast<volatile uint32_t*>(s_scan + 20);   // index of the end marker's tile, once known
  const uint32_t mbar0 = (uint32_t)__cvta_generic_to_shared(tc_smem + L.misc + 96);
  // mbarriers: a stage's MMAs are done [2], it has been read [2]; a tile buffer's pixels and row data are in place [4],
  // the buffer has been read by its last MMA [4], its row data have been read by the consumers [4]
  const uint32_t mb_done = mbar0, mb_free = mbar0 + 16, mb_meta = mbar0 + 32, mb_tile = mbar0 + 64, mb_rows = mbar0 + 96;

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
  if (K < k_min || K > k_max || K > peak_cap) return;
  const float inf = __int_as_float(0x7f800000);
  const float qnan = __int_as_float(0x7fc00000);
  int32_t* lab_img = labels + (size_t)b * plane;
  float* best_img = best ? best + (size_t)b * plane : nullptr;
  float* second_img = second ? second + (size_t)b * plane : nullptr;
  const uint32_t pk_lbo = (uint32_t)peak_cap * 16u; // bytes between core matrices along K in the peak operand
  const bool score_all = WANT2 || need_exact;       // scores wanted: every row is re-scored
  const int R1 = (K + kTcRound - 1) / kTcRound;     // rounds of 64 peaks
  const bool both = R1 == 2;                        // up to 128 peaks: the two stages together hold one round of all peaks
  const bool combined = R1 <= 2;                    // one round serves both passes
  const int n_rounds = combined ? 1 : 2 * R1;       // per tile: pass 1 rounds (S only), then pass 2 rounds (S and Delta)

  // ---- one-time set-up: tensor memory, barriers, zeroed tiles (padding k-slots must stay zero), peak operand
  if (wid == 0) {
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(s_tmem);
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst), "r"(kTcCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(mb_done + 8 * i, 1);    // the MMA commit
      mbar_init(mb_free + 8 * i, 4);    // one arrival per consumer warp
    }
    for (int i = 0; i < kTcMaxTiles; ++i) {
      mbar_init(mb_meta + 8 * i, 4);    // one arrival per producer warp
      mbar_init(mb_tile + 8 * i, 1);    // the MMA commit
      mbar_init(mb_rows + 8 * i, 4);    // one arrival per consumer warp
    }
    *s_abort = 0;
    for (int i = 0; i < 8; ++i) s_qfill[i] = 0;
    s_relcnt[0] = 0;
    s_relcnt[1] = 0;
    *s_endtile = 0xffffffffu;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < kTiles * kTileHalves / 2; i += kTcThreads) reinterpret_cast<uint32_t*>(s_tiles)[i] = 0u;
  // peak operand, K-major core matrices: row k = [-2 ex (2F), 0.., -2 ey (2F), 0..] in binary16 (the factor -2 is
  // exact); rows beyond the last peak are NaN, so that their columns never win a minimum nor pass a comparison
  {
    const int kn_r = R1 * kTcRound;
    for (int i = tid; i < kn_r * 2 * KA; i += kTcThreads) {
      const int k = i / (2 * KA), s = i - k * 2 * KA;
      const int axis = s / KA, cc = s - axis * KA;
      float v = 0.0f;
      if (k >= K) v = qnan;
      else if (cc < 2 * F) v = -2.0f * pk_img[(size_t)k * D + axis * 2 * F + cc];
      s_pk[(s >> 3) * (peak_cap * 8) + k * 8 + (s & 7)] = __float2half_rn(v);
    }
  }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  uint32_t rejected = 0, n_pairs = 0, n_rescored = 0, n_full = 0;
  TcScore<T> sc;
  sc.e_img = e_img; sc.pk_img = pk_img; sc.plane = plane; sc.F = F; sc.K = K; sc.tau = tau;
  sc.lab_img = lab_img; sc.best_img = best_img; sc.second_img = second_img; sc.status = status;

  if (wid >= 4) {
    // =============================================================================================== producers
    const int ptid = tid - 128, pw = ptid >> 5;
    const int gl = ptid >> 3, cq = ptid & 7;        // lane cq fetches channels cq, cq+8, ... of group gl, owns row ptid
    const int n_spans = (HW + kTcSpan - 1) / kTcSpan;
    const bool lab16 = ((uintptr_t)lab_img & 15u) == 0;
    const bool sc16 = best_img && ((uintptr_t)best_img & 15u) == 0 && ((uintptr_t)second_img & 15u) == 0;
    uint32_t t = 0, tdone = 0;                      // tiles issued, tiles completed
    uint32_t ring_head = 0, ring_tail = 0;          // groups taken, groups appended
    bool bad = false;                               // some producer's wait has run out: the same in all producers
    bool my_bad = false;                            // this thread's wait has run out (not yet agreed on)
    int pend_ng[3] = {0, 0, 0};                     // groups of the tiles whose copies are in flight, oldest first
    uint32_t pend_head[3] = {0, 0, 0};
    int n_pend = 0;

    auto slot_of = [&](int c) { return c >= 2 * F ? KA + (c - 2 * F) : c; };
    auto unit_ptr = [&](__half* tile, int c) {
      const int s = slot_of(c);
      return tile + (s >> 3) * (kTcRows * 8) + gl * 64 + (s & 7) * 8;
    };
    // copies of tile t (ng groups from ring position head) into buffer t % kTiles
    auto issue = [&](int ng, uint32_t head) {
      const int us = (int)(t % kTiles);
      if (!my_bad && !mbar_wait(mb_tile + 8 * us, ((t / kTiles) & 1u) ^ 1u, s_abort)) {   // its previous tile has been read
        my_bad = true;
        *s_abort = 1;
      }
      if constexpr (sizeof(T) == 2) {
        if (!my_bad && gl < ng) {
          const T* src0 = e_img + (size_t)s_ring[(head + gl) & (kTcRing - 1)] * 8;
          __half* tile = s_tiles + (size_t)us * kTileHalves;
          for (int c = cq; c < D; c += 8) {
            const uint32_t d32 = (uint32_t)__cvta_generic_to_shared(unit_ptr(tile, c));
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(d32), "l"(src0 + (size_t)c * plane));
          }
        }
        asm volatile("cp.async.commit_group;\n" ::);
      }
    };
    // everything else for tile u: norms, constants, rounds.  `newer` = copy groups issued after this tile's.
    auto complete = [&](uint32_t u, int ng, uint32_t head, int newer) {
      const int us = (int)(u % kTiles);
      __half* tile = s_tiles + (size_t)us * kTileHalves;
      float ax[8], ay[8];
#pragma unroll
      for (int r = 0; r < 8; ++r) ax[r] = ay[r] = 0.0f;
      auto add_squares = [&](const uint4& q, int c) {
        const __half2* h = reinterpret_cast<const __half2*>(&q);
        float f[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 v = __half22float2(h[i]);
          f[2 * i] = v.x;
          f[2 * i + 1] = v.y;
        }
        if (c < 2 * F) {
#pragma unroll
          for (int r = 0; r < 8; ++r) ax[r] = fmaf(f[r], f[r], ax[r]);
        } else {
#pragma unroll
          for (int r = 0; r < 8; ++r) ay[r] = fmaf(f[r], f[r], ay[r]);
        }
      };
      uint32_t grp = 0, bits = 0;
      if (gl < ng) {
        grp = s_ring[(head + gl) & (kTcRing - 1)];
        bits = s_ringbits[(head + gl) & (kTcRing - 1)];
      }
      if constexpr (sizeof(T) == 2) {
        if (newer >= 2) asm volatile("cp.async.wait_group 2;\n" ::: "memory");
        else if (newer == 1) asm volatile("cp.async.wait_group 1;\n" ::: "memory");
        else asm volatile("cp.async.wait_group 0;\n" ::: "memory");
        if (gl < ng)
          for (int c = cq; c < D; c += 8) add_squares(*reinterpret_cast<const uint4*>(unit_ptr(tile, c)), c);
      } else {
        // binary32: two 128-bit loads per unit, rounded to binary16 on the way
        if (gl < ng) {
          const T* src0 = e_img + (size_t)grp * 8;
          for (int c = cq; c < D; c += 8) {
            const float4* src = reinterpret_cast<const float4*>(src0 + (size_t)c * plane);
            const float4 lo = __ldg(src), hi = __ldg(src + 1);
            __half2 h[4] = {__floats2half2_rn(lo.x, lo.y), __floats2half2_rn(lo.z, lo.w),
                            __floats2half2_rn(hi.x, hi.y), __floats2half2_rn(hi.z, hi.w)};
            const uint4 q = *reinterpret_cast<const uint4*>(h);
            *reinterpret_cast<uint4*>(unit_ptr(tile, c)) = q;
            add_squares(q, c);
          }
        }
      }
      fence_async_smem();
      const float nx = reduce_scatter8(ax, cq), ny = reduce_scatter8(ay, cq);

      // this thread's row (pixel cq of group gl): flags, error bounds, accumulator constants
      const bool in_group = gl < ng;
      const bool present = in_group && ((bits >> cq) & 1u);
      const bool finite = (nx + ny) < inf;
      // binary16 pixels: a non-finite norm is a non-finite pixel.  binary32 pixels: it may also be a value beyond
      // the binary16 range, so the row is scored exactly (and its finiteness checked there).
      const bool live = present && finite;
      uint32_t flags = 0;
      if (in_group) flags |= kRfGroup;
      if (present) flags |= kRfPresent;
      if (live) flags |= kRfLive;
      if (present && !finite && sizeof(T) == 4) flags |= kRfHard;
      float cS, cD, dS;      // S_lo <= S <= S_lo + 2 dS and |Delta - Delta_c| <= dS
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
      // row data for the consumers (who must be through with the buffer's previous tile's); with the arrival the tile
      // is handed to the MMA warp as well
      if (!my_bad && !mbar_wait(mb_rows + 8 * us, ((u / kTiles) & 1u) ^ 1u, s_abort)) {
        my_bad = true;
        *s_abort = 1;
      }
      s_rpix[us * kTcRows + ptid] = grp * 8u + (uint32_t)cq;
      s_rslack[us * kTcRows + ptid] = dS;
      s_rcs[us * kTcRows + ptid] = cS;
      s_rcd[us * kTcRows + ptid] = cD;
      s_rflags[us * kTcRows + ptid] = flags;
      __syncwarp();
      // (`test_stall`, tests of the time-out path only: the first tile's arrival is withheld, so that the consumers'
      // bounded wait for it runs out and the CTA winds down)
      if (lane == 0 && !(test_stall && u == 0)) mbar_arrive(mb_meta + 8 * us);
    };
    // a new tile's copies go out, then the oldest tile in flight is completed once kAhead newer ones are on their way
    auto emit = [&](int ng) {
      const uint32_t head = ring_head;
      issue(ng, head);
      ring_head += (uint32_t)ng;
      pend_ng[n_pend] = ng;
      pend_head[n_pend] = head;
      ++n_pend;
      ++t;
      if (n_pend > kAhead) {
        complete(tdone, pend_ng[0], pend_head[0], n_pend - 1);
        ++tdone;
        pend_ng[0] = pend_ng[1]; pend_ng[1] = pend_ng[2];
        pend_head[0] = pend_head[1]; pend_head[1] = pend_head[2];
        --n_pend;
      }
    };

    // mask of this thread's group in a span, loaded one span ahead
    auto load_mask = [&](int sp) -> uint32_t {
      const long long p0 = (long long)(n_spans - 1 - sp) * kTcSpan + (long long)ptid * 8;
      uint32_t bits = 0;
      if (sp >= 0 && sp < n_spans && p0 < HW) {        // HW is a multiple of 8: the whole group is inside
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
      }
      return bits;
    };
    // Spans are handed out by a ticket counter (one per image, zero at launch): later spans first, because the tail
    // of the voting pass is what is still in L2, and dynamically, because the participating pixels are spread unevenly.
    uint32_t* ticket = acc + b * kAccStride + kAccSpan;
    if (ptid == 0) s_scan[6] = (int)atomicAdd(ticket, 1u);
    bad = producers_sync_or(my_bad);
    int cur = s_scan[6];
    uint32_t next_bits = load_mask(cur);
    while (cur < n_spans && !bad) {
      const long long span0 = (long long)(n_spans - 1 - cur) * kTcSpan;
      const long long p0 = span0 + (long long)ptid * 8;
      const uint32_t bits = next_bits;
      if (ptid == 0) s_scan[7] = (int)atomicAdd(ticket, 1u);    // the span after this one
      if (p0 < HW && bits == 0) {
        // a group without a participating pixel: its outputs are written here
        if (lab16) {
          reinterpret_cast<int4*>(lab_img + p0)[0] = make_int4(0, 0, 0, 0);
          reinterpret_cast<int4*>(lab_img + p0)[1] = make_int4(0, 0, 0, 0);
        } else {
          for (int j = 0; j < 8; ++j) lab_img[p0 + j] = 0;
        }
        if (best_img) {
          if (sc16) {
            const float4 v = make_float4(inf, inf, inf, inf);
            reinterpret_cast<float4*>(best_img + p0)[0] = v;
            reinterpret_cast<float4*>(best_img + p0)[1] = v;
            reinterpret_cast<float4*>(second_img + p0)[0] = v;
            reinterpret_cast<float4*>(second_img + p0)[1] = v;
          } else {
            for (int j = 0; j < 8; ++j) {
              best_img[p0 + j] = inf;
              second_img[p0 + j] = inf;
            }
          }
        }
      }
      // append the participating groups to the ring, in pixel order
      const uint32_t gm = __ballot_sync(0xffffffffu, bits != 0);
      if (lane == 0) s_scan[pw] = __popc(gm);
      bad = producers_sync_or(my_bad);
      if (bad) break;
      const int nxt = s_scan[7];
      next_bits = load_mask(nxt);                      // in flight while this span's tiles are put together
      int before = 0, total = 0;
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int v = s_scan[w];
        if (w < pw) before += v;
        total += v;
      }
      if (bits) {
        const uint32_t pos = ring_tail + (uint32_t)before + (uint32_t)__popc(gm & ((1u << lane) - 1u));
        s_ring[pos & (kTcRing - 1)] = (uint32_t)(p0 >> 3);
        s_ringbits[pos & (kTcRing - 1)] = (uint8_t)bits;
      }
      bad = producers_sync_or(my_bad);  // ring entries written, scan scratch free again
      if (bad) break;
      ring_tail += (uint32_t)total;
      while (ring_tail - ring_head >= (uint32_t)kTcGroups) emit(kTcGroups);
      cur = nxt;
    }
    if (!bad && ring_tail != ring_head) emit((int)(ring_tail - ring_head));
    while (!bad && n_pend > 0) {
      complete(tdone, pend_ng[0], pend_head[0], n_pend - 1);
      ++tdone;
      pend_ng[0] = pend_ng[1]; pend_ng[1] = pend_ng[2];
      pend_head[0] = pend_head[1]; pend_head[1] = pend_head[2];
      --n_pend;
    }
    if (!bad) {
      // end marker in the row data of the next tile buffer, once the buffer's previous tile has been worked off
      const int us = (int)(t % kTiles);
      if (!mbar_wait(mb_tile + 8 * us, ((t / kTiles) & 1u) ^ 1u, s_abort) ||
          !mbar_wait(mb_rows + 8 * us, ((t / kTiles) & 1u) ^ 1u, s_abort)) {
        my_bad = true;
        *s_abort = 1;
      }
      s_rflags[us * kTcRows + ptid] = kRfEnd;
      if (ptid == 0) *s_endtile = t;
      __syncwarp();
      if (lane == 0) mbar_arrive(mb_meta + 8 * us);
    }
    if (bad || my_bad) {
      *s_abort = 1;
      tc_timed_out(status);
    }
    asm volatile("cp.async.wait_all;\n" ::: "memory");
  } else {
    // =============================================================================================== consumers
    const uint32_t t_lane = tmem + ((uint32_t)(wid * 32) << 16);
    unsigned long long* Qw = s_queue + (size_t)wid * kTcQueue;
    uint32_t* Hw = s_hardq + (size_t)wid * kTcHardQueue;
    int qn = 0, nh = 0;                             // the warp's queue fill (the same in all lanes)
    uint32_t t = 0, rc = 0;                         // tiles taken, rounds taken
    bool bad = false;                               // a wait of this warp has run out
    // waits as a warp: either every lane saw the phase complete, or the warp gives up
    auto wait_all = [&](uint32_t mbar, uint32_t parity) {
      const bool ok = mbar_wait(mbar, parity, s_abort);
      return __all_sync(0xffffffffu, ok) != 0;
    };
    // MMAs of round q (counted over all tiles) into stage q & 1; called by one lane.  The tile's operand has to be in
    // place (its end marker stops the issue) and the stage has to have been read by all four consumer warps.
    const uint64_t da0 = tc_desc((uint32_t)__cvta_generic_to_shared(s_tiles), kTileLbo, 128u);
    const uint64_t db0 = tc_desc((uint32_t)__cvta_generic_to_shared(s_pk), pk_lbo, 128u);
    auto issue_round = [&](uint32_t q) -> bool {
      const uint32_t tq = q / (uint32_t)n_rounds;
      const int r = (int)(q - tq * (uint32_t)n_rounds);
      const int us = (int)(tq % kTiles);
      const uint32_t as = both ? 0u : (q & 1u);
      const uint32_t uses = both ? q : (q >> 1);    // how often the stage has been used before
      // wait for the tile's operand -- or for the news that the tiles ended before this one
      {
        bool ready = false;
        for (int it = 0; it < kTcWaitLimit && !ready; ++it) {
          uint32_t done;
          asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
                       : "=r"(done) : "r"(mb_meta + 8 * us), "r"((tq / kTiles) & 1u) : "memory");
          if (done) ready = true;
          else if (*s_endtile < tq) return true;
          else if ((it & 15) == 15 && *s_abort) return false;
        }
        if (!ready) return false;
      }
      if (*reinterpret_cast<volatile uint32_t*>(s_rflags + us * kTcRows) & kRfEnd) return true;
      if (!mbar_wait(mb_free + 8 * as, (uses & 1u) ^ 1u, s_abort)) return false;
      tc_fence_after();
      const bool with_delta = combined || r >= R1;
      const uint64_t da = da0 + (uint64_t)(((uint32_t)us * (kTileHalves * 2)) >> 4);
      for (int h = 0; h < (both ? 2 : 1); ++h) {     // `both`: peaks 0..63 into stage 0, 64..127 into stage 1
        const uint64_t db = db0 + (uint64_t)(((uint32_t)((r % R1 + h) * kTcRound) * 16u) >> 4);
#pragma unroll
        for (int acc = 0; acc < 2; ++acc) {
          if (acc == 1 && !with_delta) continue;
#pragma unroll
          for (int ks = 0; ks < 2 * KS; ++ks) {
            const uint32_t id = (acc == 1 && ks >= KS) ? (kTcIdesc | kTcNegB) : kTcIdesc;
            tc_mma(tmem + (as + (uint32_t)h) * 128u + (uint32_t)(acc * 64), da + (uint64_t)((ks * 2u * kTileLbo) >> 4),
                   db + (uint64_t)((ks * 2u * pk_lbo) >> 4), id, ks > 0);
          }
        }
      }
      tc_commit(mb_done + 8 * as);
      if (r == n_rounds - 1) tc_commit(mb_tile + 8 * us);
      return true;
    };
    // This warp is through with round q's stage.  The last of the four warps to say so issues round q + 2 into it.
    auto release_stage = [&](uint32_t q) {
      const uint32_t as = both ? 0u : (q & 1u);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(mb_free + 8 * as);
        const uint32_t old = atomicAdd(&s_relcnt[as], 1u);
        if ((old & 3u) == 3u && !issue_round(q + (both ? 1u : 2u))) {
          *s_abort = 1;
          tc_timed_out(status);
        }
      }
      __syncwarp();
    };
    // the first two rounds have nobody to release their stages
    if (tid == 0) {
      if (!issue_round(0) || (!both && !issue_round(1))) {
        *s_abort = 1;
        tc_timed_out(status);
      }
    }
    __syncwarp();

    while (true) {
      const int us = (int)(t % kTiles);
      if (!wait_all(mb_meta + 8 * us, (t / kTiles) & 1u)) { bad = true; break; }
      const uint32_t flags = s_rflags[us * kTcRows + tid];
      if (flags & kRfEnd) break;                    // every row of the marker carries it
      const uint32_t pix = s_rpix[us * kTcRows + tid];
      const float dS = s_rslack[us * kTcRows + tid];
      const float cS = s_rcs[us * kTcRows + tid], cD = s_rcd[us * kTcRows + tid];
      __syncwarp();
      if (lane == 0) mbar_arrive(mb_rows + 8 * us);       // the buffer's row data may be overwritten
      const bool live = (flags & kRfLive) != 0;

      // ---- pass 1: the smallest (and, if the runner-up is wanted, second smallest) S_k of the row
      float s1 = inf, s2 = inf;
      uint32_t as = 0;
      for (int r = 0; r < R1; ++r) {
        if (!both || r == 0) {
          as = both ? 0u : (rc & 1u);
          if (!wait_all(mb_done + 8 * as, (both ? rc : (rc >> 1)) & 1u)) { bad = true; break; }
          tc_fence_after();
        }
        const uint32_t st = as + (both ? (uint32_t)r : 0u);      // the stage that holds this round's columns
        const int kn = K - r * kTcRound;
        for (int c0 = 0; c0 < kTcRound && c0 < kn; c0 += 32) {
          float vS[32];
          tc_ld32(t_lane + st * 128u + (uint32_t)c0, vS);
          float bm = inf;               // the block's own minimum: pass 2 skips blocks that cannot hold a candidate
#pragma unroll
          for (int j = 0; j < 32; j += 2) bm = min3f(bm, vS[j], vS[j + 1]);   // columns beyond the last peak are NaN
          if (combined) s_bmin[(2 * r + (c0 >> 5)) * kTcRows + tid] = bm;
          if constexpr (WANT2) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float v = (vS[j] == vS[j]) ? vS[j] : inf;
              const float lo = fminf(s1, v), hi = fmaxf(s1, v);
              s1 = lo;
              s2 = fminf(s2, hi);
            }
          } else {
            s1 = fminf(s1, bm);
          }
        }
        if (!combined) {
          release_stage(rc);
          ++rc;
        }
      }
      if (bad) break;
      // d_best^2 <= 2 S_true(arg-min) <= 2 (S_lo + 2 dS).  A peak can only win if L_true <= d_best^2, and what pass 2
      // computes, 2 S_lo - |Delta_c|, is at most L_true + dS: the test is 2 S_lo - |Delta_c| <= 2 (S_min + 2 dS) + dS.
      // Rows without a usable pixel get a NaN threshold: no comparison with it is ever true.
      // The accumulators hold the dot products alone: S_lo = cS + S_acc, Delta_c = cD + Delta_acc.  The row constant
      // 2 cS is moved to the other side of the comparison (rounded up).
      const float sref = (WANT2 ? s2 : s1) + cS;
      const float thr_full = (2.0f * (sref + 2.0f * dS) * (1.0f + 1e-5f) + 1e-6f) + dS;
      const float thr = live ? (thr_full - 2.0f * cS) + 1e-5f * (fabsf(thr_full) + 2.0f * cS) : qnan;
      // |Delta_c| <= S_lo + 3 dS = cS + S_acc + 3 dS, so what pass 2 tests is at least S_acc - cS - 3 dS: a column
      // can only pass if S_acc <= thrS, and a block of 32 columns whose smallest S_acc is above it for every row of
      // the warp is not looked at again (neighbouring pixels have the same few peaks close by: most blocks go).
      const float thrS = (thr + cS + 3.0f * dS) + 1e-5f * (fabsf(thr) + cS);

      // ---- pass 2: L_k <= thr as a bit mask.  A peak that passes gets bounds dlo <= d <= dhi from its S and Delta
      // (A = (S + Delta) / 2, B = (S - Delta) / 2); the smallest dhi, U, bounds the best distance, and the candidates
      // are the peaks with dlo <= U.  (The runner-up wanted: the second smallest dhi.)
      int cnt = 0;                       // candidates appended so far
      bool lost = false;                 // some candidate has no bounds: keep them all
      float U1 = inf, U2 = inf;
      auto append = [&](int k, float dlo) {
        if (cnt < kTcCand) {
          s_cand[cnt * kTcRows + tid] = (uint16_t)k;
          s_clo[cnt * kTcRows + tid] = dlo;
        }
        ++cnt;
      };
      for (int r = 0; r < R1; ++r) {
        if (!combined) {
          as = rc & 1u;
          if (!wait_all(mb_done + 8 * as, (rc >> 1) & 1u)) { bad = true; break; }
          tc_fence_after();
        }
        const uint32_t st = as + (both ? (uint32_t)r : 0u);
        const int kn = K - r * kTcRound;
        for (int c0 = 0; c0 < kTcRound && c0 < kn; c0 += 32) {
          if (combined) {
            const bool need = live && s_bmin[(2 * r + (c0 >> 5)) * kTcRows + tid] <= thrS;
            if (!__any_sync(0xffffffffu, need)) continue;
          }
          float vS[32], vD[32];
          tc_ld32x2(t_lane + st * 128u + (uint32_t)c0, t_lane + st * 128u + 64u + (uint32_t)c0, vS, vD);
          // Four chains, one per column number mod 4: the OR into one mask would serialise the loop, and each chain
          // remembers S and Delta of its last column that passed -- so up to four columns that pass in one block of
          // 32 still have their values at hand as long as their numbers differ mod 4 (peaks next to each other in
          // the list, which are next to each other on the map, always do).
          uint32_t mq[4] = {0u, 0u, 0u, 0u};
          float xs[4] = {0.0f, 0.0f, 0.0f, 0.0f}, xd[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float d = vD[j + i] + cD;
              if (fmaf(2.0f, vS[j + i], -fabsf(d)) <= thr) { mq[i] |= 1u << (j + i); xs[i] = vS[j + i]; xd[i] = d; }
            }
          }
          const int rem = kn - c0;
          const uint32_t valid = rem < 32 ? (1u << rem) - 1u : 0xffffffffu;
#pragma unroll
          for (int i = 0; i < 4; ++i) mq[i] &= valid;
          uint32_t mk = (mq[0] | mq[1]) | (mq[2] | mq[3]);
          if (mk) {
            const int kbase = r * kTcRound + c0;
            n_pairs += (uint32_t)__popc(mk);
            while (mk) {                       // in ascending k: the list keeps that order
              const int j = __ffs(mk) - 1;
              mk &= mk - 1;
              const int i = j & 3;
              const uint32_t mi = i == 0 ? mq[0] : i == 1 ? mq[1] : i == 2 ? mq[2] : mq[3];
              if ((mi & (mi - 1)) == 0) {
                // the only one of its chain: bounds dlo <= d <= dhi from its S and Delta
                const float xs_ = i == 0 ? xs[0] : i == 1 ? xs[1] : i == 2 ? xs[2] : xs[3];
                const float xd_ = i == 0 ? xd[0] : i == 1 ? xd[1] : i == 2 ? xd[2] : xd[3];
                const float Slo = cS + xs_;
                const float e = dS + 4e-6f * (fabsf(Slo) + fabsf(xd_));           // |S - S_lo - e| <= e, |Delta - xd| <= e
                const float a_lo = 0.5f * (Slo + xd_ - e), b_lo = 0.5f * (Slo - xd_ - e);
                const float dlo = (__fsqrt_rn(fmaxf(a_lo, 0.0f)) + __fsqrt_rn(fmaxf(b_lo, 0.0f))) * (1.0f - 2e-6f);
                const float dhi = (__fsqrt_rn(fmaxf(a_lo + 2.0f * e, 0.0f)) + __fsqrt_rn(fmaxf(b_lo + 2.0f * e, 0.0f))) * (1.0f + 2e-6f);
                if (dhi < U1) { U2 = U1; U1 = dhi; }
                else if (dhi < U2) { U2 = dhi; }
                const float Uref = WANT2 ? U2 : U1;
                if (dlo <= Uref * (1.0f + 4e-5f) + 1e-6f) append(kbase + j, dlo);
              } else {
                // several of one chain: kept without bounds
                lost = true;
                append(kbase + j, 0.0f);
              }
            }
          }
        }
        if (!both || r == R1 - 1) {
          release_stage(rc);
          ++rc;
        }
      }
      if (bad) break;
      // what is left of the list once U is final (the order, ascending k, is kept)
      if (cnt <= kTcCand) {
        const float Uref = WANT2 ? U2 : U1;
        const float Um = Uref * (1.0f + 4e-5f) + 1e-6f;
        int kept = 0;
        for (int i = 0; i < cnt; ++i) {
          const float dlo = s_clo[i * kTcRows + tid];
          const uint16_t k = s_cand[i * kTcRows + tid];
          if (lost || dlo <= Um) {
            s_cand[kept * kTcRows + tid] = k;
            ++kept;
          }
        }
        cnt = kept;
      }
      if (bad) break;
      if (live) am_ok(cnt > 0, 9u, status);                 // the arg-min always passes

      // ---- the row's outcome: decided here, or queued for the scoring step
      int hard = (flags & kRfHard) ? 1 : 0;
      if (live && cnt > kTcCand) hard = 1;
      int want = 0;                                         // (kept as separate statements)
      if (live && score_all) want = 1;
      if (live && cnt > 1) want = 1;
      if (hard) want = 0;
      if (flags & kRfGroup) {
        // 8 lanes = the 8 pixels of a group: a full 32-byte sector.  Queued rows get their label when they are scored.
        int label = 0;
        if (live && !want && !hard && cnt == 1) label = (int)s_cand[tid] + 1;   // decided by the filter alone (tau = +inf, no scores)
        lab_img[pix] = label;
        if (best_img && !want && !hard) {
          best_img[pix] = inf;                              // a pixel that takes no part
          second_img[pix] = inf;
        }
      }
      {
        // queue slots: the few lanes that queue take them with an atomic on the warp's counter (the order of the
        // rows within the queue does not matter)
        const int need = want ? 1 + cnt : 0;
        if (want) {
          const int pos = atomicAdd(&s_qfill[wid], need);
          if (am_ok(pos >= 0 && pos + cnt < kTcQueue, 3u, status)) {
            const unsigned long long hi = (unsigned long long)pix << 32;
            Qw[pos] = hi | kTcHeader | (uint32_t)cnt;
            for (int i = 0; i < cnt; ++i) Qw[pos + 1 + i] = hi | (uint32_t)s_cand[i * kTcRows + tid];
            if (cnt > 1) ++n_rescored;
          }
        }
        __syncwarp();
        qn = *reinterpret_cast<volatile int*>(&s_qfill[wid]);
        const uint32_t hm = __ballot_sync(0xffffffffu, hard != 0);
        if (hard) {
          const int hp = nh + __popc(hm & ((1u << lane) - 1u));
          if (am_ok(hp < kTcHardQueue, 2u, status)) Hw[hp] = pix;
        }
        nh += __popc(hm);
        if (qn > kTcFlushAt || nh > kTcHardFlushAt) {
          tc_flush_warp<T, KA>(sc, Qw, min(qn, kTcQueue), Hw, min(nh, kTcHardQueue), 0, 1, rejected, n_full);
          qn = 0;
          nh = 0;
          if (lane == 0) s_qfill[wid] = 0;
          __syncwarp();
        }
      }
      ++t;
    }
    if (bad) {
      *s_abort = 1;
      tc_timed_out(status);
    }
    __syncwarp();
    if (lane == 0) {
      s_qfill[wid] = min(qn, kTcQueue);
      s_qfill[4 + wid] = min(nh, kTcHardQueue);
    }
  }

  // ---- every role is through: what is still queued is scored by all warps, two per queue
  tc_fence_before();
  __syncthreads();
  if (!*s_abort) {
    const int q = wid & 3, part = wid >> 2;
    tc_flush_warp<T, KA>(sc, s_queue + (size_t)q * kTcQueue, s_qfill[q], s_hardq + (size_t)q * kTcHardQueue, s_qfill[4 + q],
                         part, 2, rejected, n_full);
  }
  // ---- tear-down: tensor memory returned
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

// One launch for every image that the all-pairs kernel leaves alone: the tcgen05 pipeline where the peaks fit one
// round (there it is the faster one), the mma.sync kernel for more peaks.  The number of peaks is only known on the
// device, so the choice is made here, per image.
template <typename T, int KA, bool WANT2>
__global__ void __launch_bounds__(kTcThreads, 2)
assign_filter_kernel(const T* __restrict__ emb, const uint8_t* __restrict__ fg, int HW, int F, int K_max,
                     const float* __restrict__ peak_emb, const int32_t* __restrict__ count_ptr, float tau, int need_exact,
                     int tc_peak_cap, int tc_k_max, int tc_vec_mask, int mma_peak_cap, int mma_span, int mma_vec_mask,
                     int mma_vec_gather, int32_t* __restrict__ labels, float* __restrict__ best, float* __restrict__ second,
                     uint32_t* __restrict__ counters, uint32_t* __restrict__ status_all, uint32_t* __restrict__ votes, int cells,
                     int k_min, uint32_t* __restrict__ acc, const uint32_t* __restrict__ near_state, int test_stall) {
  static_assert(kTcThreads == kAmThreads, "both bodies run with the same block size");
  grid_dependency_sync();
  // after the pruned assignment (near_state given) this kernel only takes the images which that one handed on
  if (near_state) {
    if (blockIdx.x == 0 && threadIdx.x == 0) fold_near_counters(near_state, counters, blockIdx.y);
    if (!near_state[blockIdx.y * kNearStride + kNearGiveUp]) k_min = 0x7fffffff;
  }
  if (count_ptr[blockIdx.y] <= tc_k_max)
    assign_tc_body<T, KA, WANT2>(emb, fg, HW, F, K_max, peak_emb, count_ptr, tau, need_exact, tc_peak_cap, tc_vec_mask, labels,
                                 best, second, counters, status_all, votes, cells, k_min, tc_k_max, acc, test_stall);
  else {
    // This kernel is one that uses tensor memory: a CTA that takes the other path gives up its right to allocate at
    // once, or the SM would not take a second CTA while this one runs.
    if (threadIdx.x < 32) asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    assign_mma_body<T, KA, WANT2>(emb, fg, HW, F, K_max, peak_emb, count_ptr, tau, need_exact, mma_peak_cap, mma_span,
                                  mma_vec_mask, mma_vec_gather, labels, best, second, counters, status_all, votes, cells,
                                  max(k_min, tc_k_max + 1));
  }
}

}  // namespace cpe
