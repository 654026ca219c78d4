// Persistent, warp-specialised tensor-core kernel: all 2T half-steps of the forward pass in ONE
// launch.  One CTA per SM walks a static list of 128-row tiles ordered half-step by half-step
// (R1 of every head, L1 of every head, R2 ...).  A tile of half-step p of head h may start once
// every tile of half-step p-1 of the same head has been stored; that is tracked with one counter
// per (half-step, head) in the workspace.  Because the list is ordered and every CTA takes its tiles
// in increasing order, each dependency points to a tile some resident CTA has already taken, so the
// (bounded) waits cannot deadlock; with the phase-major order a dependency is almost a whole
// half-step old when it is needed and the waits are normally free.
//
// Warp roles (384 threads):
//   warp 0      TMA producer (one thread, polling, never blocking): checks the tile's dependency
//               counter (fetched one tile ahead) and loads its operands into three rings
//               (E: operand released after MMA 1, L: operand released after MMA 2, V: V/y tile)
//   warp 1      MMA issuer: scores S = A.B^T into TMEM (two accumulator stages), then, once the
//               softmax group has written P to shared memory, the apply MMA into O
//   warps 2-5   softmax group 0 (tiles 0, 2, 4, ... of this CTA): one thread per score row
//   warps 6-9   softmax group 1 (tiles 1, 3, 5, ...)
//   warps 10,11 store threads (one per softmax group, in warps of their own because a suspended
//               mbarrier wait suspends the whole warp): TMA-store the staged rows, wait until
//               they are in global memory, then bump the (half-step, head) counter
// No role ever waits for another CTA while holding up work of an earlier tile of its own CTA: the
// MMA issuer polls its two pending jobs (MMA 2 of the oldest tile, MMA 1 of the next) instead of
// blocking on either, and completion is signalled by the store lanes, not by the softmax groups.
// A softmax group reads S from TMEM (two passes: row max, then exp/sum), writes P (16-bit,
// 128-byte swizzled) for MMA 2, later reads O from TMEM, normalises, stages the 16-bit rows in the
// same buffer and one thread TMA-stores them with the strides that realise the permutation.
#pragma once
#include "tensor_path.cuh"

namespace ma {
namespace tp {

using namespace ma::tensor;

constexpr int kThreads = 384;
constexpr int kRingE = 2, kRingL = 4, kRingV = 3;
constexpr int kSlot = kTileBytes;   // 16 KB

struct Lay {
  static constexpr int E = 0;
  static constexpr int L = E + kRingE * kSlot;
  static constexpr int V = L + kRingL * kSlot;
  static constexpr int P = V + kRingV * kSlot;          // 2 x 32 KB
  static constexpr int Ones = P + 4 * kSlot;            // 2 KB
  static constexpr int Vec = Ones + 2048;               // kRingL x 128 floats (c_R / c_L)
  static constexpr int Bars = Vec + kRingL * 512;
  static constexpr int Total = Bars + 256;
};
constexpr int kSmem = Lay::Total + 1024;

struct __align__(8) Bars {
  uint64_t fullE[kRingE], emptyE[kRingE];
  uint64_t fullL[kRingL], emptyL[kRingL];
  uint64_t fullV[kRingV], emptyV[kRingV];
  uint64_t s_ready[2], p_half[2], p_ready[2], o_ready[2], o_free[2], stage_ready[2], stage_free[2];
  uint32_t tmem_slot;
  volatile int abort_flag;
  long long wait_limit;   // clocks a wait may take before it gives up
};

struct Params {
  CUtensorMap tmQ, tmK, tmV, tmAR, tmAL, tmY;    // 2D row views (loads)
  CUtensorMap tmALs, tmYs;                       // 3D stores of aL / y (rows m apart)
  CUtensorMap tmQs;                              // 3D strided view of Q (load)
  CUtensorMap tmARs, tmOut;                      // 3D strided stores of aR / Y
  CUtensorMap tmALlo, tmALlos;                   // low halves of alpha_L (second-generation kernel, bf16, b = 32)
  float* cL;
  float* cR;
  uint8_t *aL, *aR, *y;  // state arrays (for L2 discards once a tile has been consumed)
  uint8_t* out;         // Y
  float* lse;           // optional [BH][N]: log-sum-exp of each row of the final L half-step
  int* status;
  int* counters;       // [2T][BH] completed tiles
  long long* trace;    // optional: clock64 stamps [4 CTAs][64 tiles][8 events] (profiling aid)
  int m, BH, T;
  int H;               // 0: Q, K, V, Y are [batch][heads][N][d]; heads: [batch][N][heads][d]
  int n_valid;         // 0: no padding; else keys b k + i >= n_valid are masked (second generation, SB == B)
  int tiles_per_head, tiles_per_phase;
  int g_begin, g_end;  // tile range of this launch
  int check_deps;
  int n_counters;      // 2T * BH
  long long wait_cycles;
  float scale;
};

struct Tile {
  int p, h, idx0;      // half-step, head, first k (R) or j (L) of the tile
  bool isR, first, withV, final_;
};
// Walks the tiles g0, g0 + step, g0 + 2 step, ... of one role without integer divisions
// (tiles_per_head is a power of two on this path).
struct TileIter {
  int p, local, step, tpp, tph_shift, tph_mask, kTiles, lastR;
  __device__ __forceinline__ TileIter(const Params& P, int g0, int step_, int kTiles_)
      : step(step_), tpp(P.tiles_per_phase), kTiles(kTiles_), lastR(2 * P.T - 2) {
    p = g0 / tpp;
    local = g0 - p * tpp;
    tph_shift = 31 - __clz(P.tiles_per_head);
    tph_mask = P.tiles_per_head - 1;
  }
  __device__ __forceinline__ Tile get() const {
    Tile t;
    t.p = p;
    t.h = local >> tph_shift;
    t.idx0 = (local & tph_mask) * kTiles;
    t.isR = (p & 1) == 0;
    t.first = p == 0;
    t.withV = p == lastR;
    t.final_ = p == lastR + 1;
    return t;
  }
  __device__ __forceinline__ void next() {
    local += step;
    while (local >= tpp) { local -= tpp; ++p; }
  }
};

// Bounded wait.  A wait that runs out records where in the status word and raises the CTA's abort
// flag; from then on every wait of the CTA returns at once, so all roles run through their
// remaining (now meaningless) tiles without blocking, barriers stay matched, and the kernel ends.
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, Bars* bars,
                                              int* status, int where) {
  const uint32_t addr = smem_u32(bar);
  const long long t0 = clock64();
  for (;;) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(addr), "r"(parity)
        : "memory");
    if (done) return true;
    if (bars->abort_flag) return false;
    if (clock64() - t0 > bars->wait_limit) {
      report_timeout(status, where);
      bars->abort_flag = 1;
      return false;
    }
  }
}
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return done != 0;
}
// Profiling aid: CTAs 0-3 stamp eight pipeline events of their first 64 tiles.
__device__ __forceinline__ void stamp(const Params& P, int n, int ev) {
  if (P.trace != nullptr && blockIdx.x < 4 && n < 64)
    P.trace[((size_t)blockIdx.x * 64 + n) * 8 + ev] = clock64();
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void group_barrier(int id) {
  asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory");
}
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void tma_store_commit() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_all() {
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
// 1-D bulk copy global -> shared (16-byte aligned, size a multiple of 16), completes on `bar`.
__device__ __forceinline__ void bulk_load_1d(void* dst, const void* src, uint32_t bytes,
                                             uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ float tmem_ld1(uint32_t taddr) {
  uint32_t r;
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r) : "r"(taddr) : "memory");
  return __uint_as_float(r);
}

// B  = rows of one MMA tile (64 or 128); SB = the method's block size b = m (SB divides B).
// With SB < B an MMA tile holds B / SB independent blocks on its diagonal: a score row only owns
// the SB columns of its own block, the other columns of P are written as zeros, and the MMAs run
// unchanged (b = 32 on M = 64 tiles wastes half the tensor work but none of the exponentials).
template <typename T, int B, int SB>
__global__ void __launch_bounds__(kThreads, 1) monarch_persistent(const __grid_constant__ Params P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  Bars* bars = reinterpret_cast<Bars*>(smem + Lay::Bars);
  constexpr int kBlocks = kRows / SB;         // blocks (k of an R tile, j of an L tile) per CTA
  constexpr int NSUB = B / SB;                // blocks per MMA tile
  // P and the states alpha_L, alpha_R, y have the inputs' type: kind::f16 needs A and B in the
  // SAME 16-bit format on this hardware (an f16 operand against a bf16 one is an illegal
  // instruction, although the instruction descriptor has a format field for each).
  typedef T S;
  constexpr int FT = Fmt<T>::code, FS = Fmt<S>::code;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m = P.m;

  if (tid == 0) {
    for (int i = 0; i < kRingE; ++i) { mbar_init(&bars->fullE[i], 1); mbar_init(&bars->emptyE[i], 1); }
    for (int i = 0; i < kRingL; ++i) { mbar_init(&bars->fullL[i], 1); mbar_init(&bars->emptyL[i], 1); }
    for (int i = 0; i < kRingV; ++i) { mbar_init(&bars->fullV[i], 1); mbar_init(&bars->emptyV[i], 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->s_ready[i], 1);
      mbar_init(&bars->p_half[i], 128);
      mbar_init(&bars->p_ready[i], 128);
      mbar_init(&bars->o_ready[i], 1);
      mbar_init(&bars->o_free[i], 128);
      mbar_init(&bars->stage_ready[i], 128);
      mbar_init(&bars->stage_free[i], 1);
    }
    bars->abort_flag = 0;
    bars->wait_limit = P.wait_cycles;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (tid < 128) {   // tile of ones for the column-sum MMA of the non-final L half-step
    const uint32_t one2 = pack2<S>(1.f, 1.f);
    *reinterpret_cast<uint4*>(smem + Lay::Ones + tid * 16) = make_uint4(one2, one2, one2, one2);
  }
  if (warp == 0) tmem_alloc(&bars->tmem_slot, 512);
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_slot;

  const int first_g = P.g_begin + blockIdx.x;
  const int stride_g = gridDim.x;
  const int n_total = first_g < P.g_end ? (P.g_end - first_g + stride_g - 1) / stride_g : 0;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const bool deps = P.check_deps != 0;
      auto counter_of = [&](const Tile& t) { return P.counters + (t.p - 1) * P.BH + t.h; };
      auto needs_v = [&](const Tile& t) { return t.isR ? t.withV : t.final_; };
      int nE = 0, nVt = 0, nv = 0;                 // next tile for E/L, next tile to scan for V
      TileIter itE(P, first_g, stride_g, kBlocks), itV(P, first_g, stride_g, kBlocks);
      while (nVt < n_total && !needs_v(itV.get())) { ++nVt; itV.next(); }
      // dependency counters are read one step ahead so their latency is off the critical path
      const uint64_t pol_first = policy_evict_first();
      int ctrE = 0, ctrV = 0;
      if (deps && nE < n_total && itE.get().p > 0) ctrE = ld_acquire(counter_of(itE.get()));
      if (deps && nVt < n_total && itV.get().p > 0) ctrV = ld_acquire(counter_of(itV.get()));
      long long t0 = clock64();
      bool force = false;
      while (nE < n_total || nVt < n_total) {
        bool did = false;
        if (nE < n_total) {
          const Tile t = itE.get();
          const int eE = nE % kRingE, eL = nE % kRingL;
          bool ok = force || !deps || t.p == 0 || ctrE >= P.tiles_per_head;
          if (!ok) { ctrE = ld_acquire(counter_of(t)); ok = ctrE >= P.tiles_per_head; }
          if (ok && (force || (mbar_test(&bars->emptyE[eE], ((nE / kRingE) & 1) ^ 1) &&
                               mbar_test(&bars->emptyL[eL], ((nE / kRingL) & 1) ^ 1)))) {
            asm volatile("fence.proxy.async.global;" ::: "memory");
            uint8_t* sE = smem + Lay::E + eE * kSlot;
            uint8_t* sL = smem + Lay::L + eL * kSlot;
            // c_R rows [k0 .. k0+kTiles) (R, not first) or c_L rows [j0 .. j0+kTiles) (L): 128 floats
            const bool needC = !t.first;
            float* sC = reinterpret_cast<float*>(smem + Lay::Vec) + eL * 128;
            mbar_expect_tx(&bars->fullE[eE], kSlot);
            mbar_expect_tx(&bars->fullL[eL], kSlot + (needC ? 512 : 0));
            if (t.isR) {
              const int row0 = (t.h * m + t.idx0) * SB;
              if (needC) bulk_load_1d(sC, P.cR + row0, 512, &bars->fullL[eL]);
              tma_load_2d(sE, t.first ? &P.tmQ : &P.tmAR, &bars->fullE[eE], 0, row0);
              tma_load_2d(sL, &P.tmK, &bars->fullL[eL], 0, row0);
            } else {
              const int row0 = (t.h * SB + t.idx0) * m;
              bulk_load_1d(sC, P.cL + row0, 512, &bars->fullL[eL]);
              tma_load_2d(sE, &P.tmAL, &bars->fullE[eE], 0, row0);
#pragma unroll
              for (int tt = 0; tt < kBlocks; ++tt)
                tma_load_3d(sL + tt * (SB * 128), &P.tmQs, &bars->fullL[eL], 0, t.idx0 + tt, t.h * m);
            }
            stamp(P, nE, 0);
            ++nE;
            itE.next();
            if (deps && nE < n_total && itE.get().p > 0) ctrE = ld_acquire(counter_of(itE.get()));
            did = true;
          }
        }
        if (nVt < n_total) {
          // the V (last R half-step) or y (last L half-step) tile is needed only by MMA 2
          const Tile t = itV.get();
          const int eV = nv % kRingV;
          bool ok = force || !deps || t.p == 0 || ctrV >= P.tiles_per_head;
          if (!ok) { ctrV = ld_acquire(counter_of(t)); ok = ctrV >= P.tiles_per_head; }
          if (ok && (force || mbar_test(&bars->emptyV[eV], ((nv / kRingV) & 1) ^ 1))) {
            asm volatile("fence.proxy.async.global;" ::: "memory");
            uint8_t* sV = smem + Lay::V + eV * kSlot;
            mbar_expect_tx(&bars->fullV[eV], kSlot);
            if (t.isR) tma_load_2d_hint(sV, &P.tmV, &bars->fullV[eV], 0, (t.h * m + t.idx0) * SB, pol_first);
            else tma_load_2d(sV, &P.tmY, &bars->fullV[eV], 0, (t.h * SB + t.idx0) * m);
            ++nv;
            do { ++nVt; itV.next(); } while (nVt < n_total && !needs_v(itV.get()));
            if (deps && nVt < n_total && itV.get().p > 0) ctrV = ld_acquire(counter_of(itV.get()));
            did = true;
          }
        }
        if (did) {
          t0 = clock64();
        } else if (!force) {
          if (bars->abort_flag) {
            force = true;
          } else if (clock64() - t0 > P.wait_cycles) {
            report_timeout(P.status, 10);
            bars->abort_flag = 1;
            force = true;
          }
          __nanosleep(32);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // Two pending jobs are polled, never waited for: MMA 2 of the oldest unfinished tile (needs P
    // from its softmax group) and MMA 1 of the next tile (needs its operands, which may depend on
    // other CTAs).  Blocking on the second would hold up the first and could deadlock the grid.
    if (elect_one()) {
      const uint32_t sE0 = smem_u32(smem + Lay::E), sL0 = smem_u32(smem + Lay::L);
      const uint32_t sV0 = smem_u32(smem + Lay::V), sP0 = smem_u32(smem + Lay::P);
      const uint32_t sOnes = smem_u32(smem + Lay::Ones);
      int i1 = 0, i2 = 0, nv = 0;
      bool half_done = false;
      TileIter it1(P, first_g, stride_g, kBlocks), it2(P, first_g, stride_g, kBlocks);
      long long t0 = clock64();
      bool force = false;
      while (i2 < n_total) {
        bool did = false;
        if (i2 < i1) {
          const Tile t = it2.get();
          const int a = i2 & 1, q = i2 >> 1, eL = i2 % kRingL;
          const bool needV = t.isR ? t.withV : t.final_;
          const int eV = nv % kRingV;
          const bool split = t.isR || t.final_;     // P arrives in two column halves
          const uint32_t sL = sL0 + eL * kSlot, sV = sV0 + eV * kSlot, sP = sP0 + a * 2 * kSlot;
          const uint32_t tO = tmem + a * 256 + 128;
          if (split && !half_done &&
              (force || (mbar_test(&bars->p_half[a], q & 1) && mbar_test(&bars->o_free[a], (q & 1) ^ 1) &&
                         (!needV || mbar_test(&bars->fullV[eV], (nv / kRingV) & 1))))) {
            // first half of the P columns is in shared memory: start MMA 2 under the softmax
            tc_fence_after();
            if (t.isR) issue_apply<B, FS, 1, FT>(tO, sP, sL, needV ? (sV - sL) : 16, needV ? 2 : 1);
            else issue_apply<B, FS, 1, FS>(tO, sP, sV, 16, 1);
            half_done = true;
            did = true;
          }
          if ((half_done || !split) &&
              (force || (mbar_test(&bars->p_ready[a], q & 1) &&
                         (split || mbar_test(&bars->o_free[a], (q & 1) ^ 1))))) {
            tc_fence_after();
            if (t.isR) {
              // [aL | y] = P [K | V]; the V tile sits (sV - sL) bytes after the K tile
              issue_apply<B, FS, 2, FT>(tO, sP, sL, needV ? (sV - sL) : 16, needV ? 2 : 1);
            } else if (t.final_) {
              issue_apply<B, FS, 2, FS>(tO, sP, sV, 16, 1);
            } else {
              issue_transposed_apply<B, FS, FT>(tO, sP, sL, sOnes);
            }
            umma_commit(&bars->emptyL[eL]);
            if (needV) { umma_commit(&bars->emptyV[eV]); ++nv; }
            umma_commit(&bars->o_ready[a]);
            stamp(P, i2, 4);
            ++i2;
            it2.next();
            half_done = false;
            did = true;
          }
        }
        if (i1 < n_total && i1 < i2 + 2) {
          const int eE = i1 % kRingE, eL = i1 % kRingL, a = i1 & 1;
          if (force || (mbar_test(&bars->fullE[eE], (i1 / kRingE) & 1) &&
                        mbar_test(&bars->fullL[eL], (i1 / kRingL) & 1))) {
            const Tile t = it1.get();
            tc_fence_after();
            const uint32_t sE = sE0 + eE * kSlot, sL = sL0 + eL * kSlot;
            // R: A = aR (E ring), B = K (L ring).  L: A = Qb (L ring), B = aL (E ring).
            if (t.isR) {
              if (t.first) issue_scores<B, FT, FT>(tmem + a * 256, sE, sL);   // A = Q
              else issue_scores<B, FS, FT>(tmem + a * 256, sE, sL);           // A = alpha_R
            } else {
              issue_scores<B, FT, FS>(tmem + a * 256, sL, sE);                // A = Qb, B = alpha_L
            }
            umma_commit(&bars->emptyE[eE]);
            umma_commit(&bars->s_ready[a]);
            stamp(P, i1, 1);
            ++i1;
            it1.next();
            did = true;
          }
        }
        if (did) {
          t0 = clock64();
        } else if (!force) {
          if (bars->abort_flag) {
            force = true;
          } else if (clock64() - t0 > P.wait_cycles) {
            report_timeout(P.status, 20);
            bars->abort_flag = 1;
            force = true;
          }
          __nanosleep(20);
        }
      }
    }
  } else if (warp < 10) {
    // ------------------------------------------------------------------ softmax groups
    const int w = (warp - 2) >> 2;             // group = accumulator stage
    const int sub = warp & 3;                  // TMEM sub-partition this warp may access
    const int t_row = sub * 32 + lane;         // TMEM lane = score row owned by this thread
    const int tile = Geo<B>::tile(t_row), r = Geo<B>::row(t_row), srow = tile * B + r;
    const int sb = r / SB, rb = r - sb * SB;     // block inside the MMA tile, row inside the block
    const int blk = tile * NSUB + sb;            // block inside the CTA's 128 rows
    const uint32_t tS = tmem + w * 256 + ((uint32_t)(sub * 32) << 16);
    const uint32_t tO = tS + 128;
    uint8_t* sP = smem + Lay::P + w * 2 * kSlot;

    TileIter it(P, first_g + w * stride_g, 2 * stride_g, kBlocks);
    for (int n = w; n < n_total; n += 2, it.next()) {
      const Tile t = it.get();
      const int q = n >> 1, eL = n % kRingL;
      const float* cv = reinterpret_cast<const float*>(smem + Lay::Vec) + eL * 128;
      // S is in tensor memory; the c-vector travelled with MMA 1's operands, whose arrival the MMA
      // thread observed before it issued (and committed) the MMA this barrier reports
      wait_or_abort(&bars->s_ready[w], q & 1, bars, P.status, 30);
      tc_fence_after();
      if (lane == 0 && sub == 0) stamp(P, n, 2);
      // MMA 1 has consumed the state tile (alpha_R rows of an R half-step, alpha_L rows of an L
      // half-step): every such tile is read exactly once, so its lines are dropped from L2 instead
      // of being written back to HBM later.
      if (t.isR) {
        if (!t.first) discard_line(P.aR + ((size_t)(t.h * m + t.idx0) * SB + t_row) * 128);
      } else {
        discard_line(P.aL + ((size_t)(t.h * SB + t.idx0) * m + t_row) * 128);
      }

      // The row is walked in 32-column chunks read from tensor memory, the next chunk being
      // fetched while the current one is processed, so that a row never has to sit in registers.
      // Arithmetic runs on packed fp32 pairs; exponentials are ex2 with log2(e) folded in.
      constexpr int NC = B / 32;
      // chunk c holds columns of this row's own block (always, when a block fills the MMA tile)
      auto mine = [&](int c) { return SB == B || (32 * c) / SB == sb; };
      float buf[32];
      float f, inv_s, mx, sum, sz = 0.f;
      size_t crow = 0;
      float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      float2 a2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      const float* cvt = cv + blk * SB;        // L: -c_L[j, :] in log2 units for this row's block
      if (t.isR) {
        // Z_R = scale * S / c_R (Eq. 7); c_L = sum R log R (Eq. 10)
        float inv_c = 1.f;
        if (!t.first) {
          const float c = cv[srow];
          inv_c = c > 1e-30f ? 1.f / c : 0.f;
        }
        f = P.scale * inv_c * kLog2e;
        crow = ((size_t)t.h * SB + rb) * m + t.idx0 + blk;     // c_L is stored [h][j][k]
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          if (!mine(c)) continue;
          tmem_ld32(tS + 32 * c, buf);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i)
            m4[i & 3] = max3(m4[i & 3], buf[2 * i], buf[2 * i + 1]);
        }
        mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        const float2 f2 = make_float2(f, f), off2 = make_float2(-mx * f, -mx * f);
        float2 z2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
        // P and the store staging share a buffer: the previous tile's rows must have been read
        wait_or_abort(&bars->stage_free[w], (q & 1) ^ 1, bars, P.status, 33);
        if (lane == 0 && sub == 0) stamp(P, n, 7);
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          float* s = buf;
          if (mine(c)) {
          tmem_ld32(tS + 32 * c, buf);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float2 sv = make_float2(s[2 * i], s[2 * i + 1]);
            const float2 zz = ffma2(sv, f2, off2);
            const float2 pp = exp2_pair(zz, i);
            z2[i & 1] = ffma2(pp, sv, z2[i & 1]);
            a2[i & 1] = fadd2(a2[i & 1], pp);
            s[2 * i] = pp.x;
            s[2 * i + 1] = pp.y;
          }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) s[i] = 0.f;
          }
          store_row32<S>(sP, srow, 32 * c, s);
          if (c == NC / 2 - 1) {    // first half of the row's P is written: MMA 2 may start on it
            fence_proxy_async();
            mbar_arrive(&bars->p_half[w]);
          }
        }
        sum = (a2[0].x + a2[0].y) + (a2[1].x + a2[1].y);
        sz = (z2[0].x + z2[0].y) + (z2[1].x + z2[1].y);
        inv_s = 1.f / sum;
      } else {
        // Z_L = scale * S' - c_L (Eq. 8), softmax over k = along the row
        f = P.scale * kLog2e;
        const float2 f2 = make_float2(f, f);
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          if (!mine(c)) continue;
          tmem_ld32(tS + 32 * c, buf);
          tmem_ld_wait();
          const float4* cv4 = reinterpret_cast<const float4*>(cvt + 32 * c - sb * SB);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float4 cc = cv4[i];
            const float2 za = ffma2(make_float2(buf[4 * i], buf[4 * i + 1]), f2,
                                    make_float2(cc.x, cc.y));
            const float2 zb = ffma2(make_float2(buf[4 * i + 2], buf[4 * i + 3]), f2,
                                    make_float2(cc.z, cc.w));
            m4[0] = max3(m4[0], za.x, za.y);
            m4[1] = max3(m4[1], zb.x, zb.y);
          }
        }
        mx = fmaxf(m4[0], m4[1]);
        const float2 nmx2 = make_float2(-mx, -mx);
        wait_or_abort(&bars->stage_free[w], (q & 1) ^ 1, bars, P.status, 33);
        if (lane == 0 && sub == 0) stamp(P, n, 7);
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          float* s = buf;
          if (mine(c)) {
          tmem_ld32(tS + 32 * c, buf);
          tmem_ld_wait();
          const float4* cv4 = reinterpret_cast<const float4*>(cvt + 32 * c - sb * SB);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float4 cc = cv4[i];
            float2 za = ffma2(make_float2(s[4 * i], s[4 * i + 1]), f2, make_float2(cc.x, cc.y));
            float2 zb = ffma2(make_float2(s[4 * i + 2], s[4 * i + 3]), f2, make_float2(cc.z, cc.w));
            za = fadd2(za, nmx2);
            zb = fadd2(zb, nmx2);
            const float2 pa = exp2_pair(za, 2 * i);
            const float2 pb = exp2_pair(zb, 2 * i + 1);
            a2[0] = fadd2(a2[0], pa);
            a2[1] = fadd2(a2[1], pb);
            s[4 * i] = pa.x;
            s[4 * i + 1] = pa.y;
            s[4 * i + 2] = pb.x;
            s[4 * i + 3] = pb.y;
          }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) s[i] = 0.f;
          }
          store_row32<S>(sP, srow, 32 * c, s);
          if (c == NC / 2 - 1 && t.final_) {    // first half of the row's P is written: MMA 2 may start on it
            fence_proxy_async();
            mbar_arrive(&bars->p_half[w]);
          }
        }
        sum = (a2[0].x + a2[0].y) + (a2[1].x + a2[1].y);
        inv_s = 1.f / sum;
        if (!t.final_) {
          // MMA 2 of this half-step contracts over rows, so P must be normalised before the MMA
          // reads it: the thread re-reads its own row, rescales it in fp32 and writes it back
          // (no other thread touches the row in between).
          const float2 is2 = make_float2(inv_s, inv_s);
#pragma unroll
          for (int c8 = 0; c8 < B / 8; ++c8) {       // 8 columns = one 16-byte chunk
            uint4* ptr = reinterpret_cast<uint4*>(sP + (c8 >> 3) * kTileBytes + srow * 128 +
                                                  (((c8 & 7) ^ (srow & 7)) << 4));
            uint4 qv = *ptr;
            uint32_t* qp = reinterpret_cast<uint32_t*>(&qv);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 v = fmul2(unpack2<S>(qp[e]), is2);
              qp[e] = pack2<S>(v.x, v.y);
            }
            *ptr = qv;
          }
        }
      }
      fence_proxy_async();
      tc_fence_before();
      if (!t.isR && !t.final_) mbar_arrive(&bars->p_half[w]);   // keeps the barrier's phase in step
      mbar_arrive(&bars->p_ready[w]);
      if (lane == 0 && sub == 0) stamp(P, n, 3);
      // -c_L in log2 units, ready to be the addend of the next L half-step's logits
      if (t.isR) P.cL[crow] = fast_log2(sum) - f * (sz * inv_s - mx);

      wait_or_abort(&bars->o_ready[w], q & 1, bars, P.status, 31);
      tc_fence_after();
      if (lane == 0 && sub == 0) stamp(P, n, 5);
      if (t.final_) discard_line(P.y + ((size_t)(t.h * SB + t.idx0) * m + t_row) * 128);   // y: read once
      const int nco = (t.isR && t.withV) ? 4 : 2;            // 32-column chunks of O
      const bool scaled = t.isR || t.final_;
      float c1 = 0.f;
      if (!t.isR && !t.final_) c1 = tmem_ld1(tO + 64);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        if (c < nco) {
          tmem_ld32(tO + 32 * c, buf);
          tmem_ld_wait();
          if (t.final_) store_row32<T>(sP, srow, 32 * c, buf, inv_s);       // Y: the caller's type
          else if (scaled) store_row32<S>(sP, srow, 32 * c, buf, inv_s);
          else store_row32<S>(sP, srow, 32 * c, buf);
        }
      }
      tc_fence_before();
      mbar_arrive(&bars->o_free[w]);
      if (!t.isR && !t.final_) P.cR[((size_t)t.h * m + rb) * SB + t.idx0 + blk] = c1;
      fence_proxy_async();
      mbar_arrive(&bars->stage_ready[w]);
      if (lane == 0 && sub == 0) stamp(P, n, 6);
    }
  } else {
    // ------------------------------------------------------------------ store threads
    if (lane == 0) {
      const int w = warp - 10;
      const uint8_t* sP = smem + Lay::P + w * 2 * kSlot;
      const uint64_t pol_first = policy_evict_first();
      TileIter it(P, first_g + w * stride_g, 2 * stride_g, kBlocks);
      for (int n = w; n < n_total; n += 2, it.next()) {
        const Tile t = it.get();
        const int q = n >> 1;
        wait_or_abort(&bars->stage_ready[w], q & 1, bars, P.status, 40);
#pragma unroll
        for (int tt = 0; tt < kBlocks; ++tt) {
          const uint8_t* src = sP + tt * (SB * 128);
          if (t.isR) {
            tma_store_3d(&P.tmALs, src, 0, t.idx0 + tt, t.h * SB);
            if (t.withV) tma_store_3d(&P.tmYs, src + kSlot, 0, t.idx0 + tt, t.h * SB);
          } else {
            if (t.final_) tma_store_3d_hint(&P.tmOut, src, 0, t.idx0 + tt, t.h * m, pol_first);
            else tma_store_3d(&P.tmARs, src, 0, t.idx0 + tt, t.h * m);
          }
        }
        tma_store_commit();
        tma_store_wait_read();
        mbar_arrive(&bars->stage_free[w]);
        tma_store_wait_all();                 // rows (and the group's c_L / c_R) are in global memory
        asm volatile("fence.proxy.async.global;" ::: "memory");
        __threadfence();
        atomicAdd(P.counters + t.p * P.BH + t.h, 1);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (bars->abort_flag) {
    // give copies still in flight time to land before shared and tensor memory are released
    const long long t0 = clock64();
    while (clock64() - t0 < 200000) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 0) tmem_dealloc(tmem, 512);
  // The last CTA to finish re-arms the dependency counters (every CTA has done its last counter
  // read by now), so that a caller who keeps the workspace need not clear it between calls.
  if (tid == 0) {
    __threadfence();
    if (atomicAdd(P.status + 1, 1) == (int)gridDim.x - 1) {
      for (int i = 0; i < P.n_counters; ++i) P.counters[i] = 0;
      P.status[1] = 0;
    }
  }
}

// ------------------------------------------------------------------------------------ host side
// Test knobs (process-wide): bound of the device-side waits, and a switch that leaves the first
// half-step out of a single-launch run so that every dependency wait of the second runs out.
struct DebugKnobs {
  long long wait_cycles = kWaitCycles;
  int skip_first_half_step = 0;
};
inline DebugKnobs& knobs() {
  static DebugKnobs k;
  return k;
}
inline long long*& trace_buffer() {
  static long long* p = nullptr;
  return p;
}
// f16/bf16, d = 64, m = b in {32, 64, 128} (b = 32 runs on 64-row MMA tiles, two blocks per tile).
inline bool supported(int N, int d, int b, int m, int dtype, int BH) {
  if (dtype != 1 && dtype != 2) return false;
  if (d != kD || b != m) return false;
  if (b != 32 && b != 64 && b != 128) return false;
  if ((long long)BH * N >= (1LL << 31)) return false;
  return true;
}
inline size_t counters_bytes(int BH, int T) {
  return ((size_t)2 * T * BH * sizeof(int) + 255) / 256 * 256;
}
// bf16 with b = 32 keeps alpha_L as a hi + lo pair of 16-bit arrays (see tensor_decoupled.cuh).
inline bool uses_hilo(int dtype, int b) { return dtype == 2 && b == 32; }
inline size_t hilo_bytes(int BH, int N) { return ((size_t)BH * N * kD * 2 + 255) / 256 * 256; }
inline size_t workspace_bytes(int BH, int N, int T, bool hilo) {
  return ws_layout(nullptr, BH, N).bytes + counters_bytes(BH, T) + (hilo ? hilo_bytes(BH, N) : 0);
}

// Defined in tensor_decoupled.cuh (the second-generation kernel, same Params).
template <typename T, int B, int SB>
cudaError_t launch_decoupled(const Params& P, int grid, cudaStream_t st);

template <typename T, int B, int SB>
inline int launch_t(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int T_steps,
                    int dtype, float scale, void* ws, cudaStream_t st, int* launches, int mode,
                    bool ws_armed, int H, float* lse, int n_valid) {
  // other layout, row log-sum-exp and the padding mask: second-generation kernel only; the mask
  // only where a tile row owns a whole key block
  if ((H != 0 || lse != nullptr || n_valid != 0) && mode != 0) return 4;
  if (n_valid != 0 && SB != B) return 4;
  const Ws w = ws_layout(ws, BH, N);
  int* counters = (int*)((char*)ws + w.bytes);
  const int m = N / SB;            // = SB on this path
  const uint64_t rows = (uint64_t)BH * N;
  void* aLlo = (char*)counters + counters_bytes(BH, T_steps);   // used when uses_hilo(dtype, SB)
  Params P;
  bool ok = make_map_rows_io(&P.tmQ, dtype, (void*)Q, rows, H) &&
            make_map_rows_io(&P.tmK, dtype, (void*)K, rows, H) &&
            make_map_rows_io(&P.tmV, dtype, (void*)V, rows, H) && make_map_rows(&P.tmAR, dtype, w.aR, rows) &&
            make_map_rows(&P.tmAL, dtype, w.aL, rows) && make_map_rows(&P.tmY, dtype, w.y, rows) &&
            true;
  constexpr uint32_t kBlk = kRows / SB;     // blocks per tile
  if (ok && mode == 0) {   // second-generation kernel: one box per tile (blocked views)
    ok = make_map_blocked_io(&P.tmALs, dtype, w.aL, m, (uint64_t)BH * SB, SB, kBlk, 0) &&
         make_map_blocked_io(&P.tmYs, dtype, w.y, m, (uint64_t)BH * SB, SB, kBlk, 0) &&
         make_map_blocked_io(&P.tmQs, dtype, (void*)Q, SB, (uint64_t)BH * m, SB, kBlk, H) &&
         make_map_blocked_io(&P.tmARs, dtype, w.aR, SB, (uint64_t)BH * m, SB, kBlk, 0) &&
         make_map_blocked_io(&P.tmOut, dtype, Y, SB, (uint64_t)BH * m, SB, kBlk, H);
    if (ok && uses_hilo(dtype, SB))
      ok = make_map_rows(&P.tmALlo, dtype, aLlo, rows) &&
           make_map_blocked_io(&P.tmALlos, dtype, aLlo, m, (uint64_t)BH * SB, SB, kBlk, 0);
  } else if (ok) {         // first-generation kernel: one box per block
    ok = make_map_strided(&P.tmALs, dtype, w.aL, m, (uint64_t)BH * SB, SB) &&
         make_map_strided(&P.tmYs, dtype, w.y, m, (uint64_t)BH * SB, SB) &&
         make_map_strided(&P.tmQs, dtype, (void*)Q, SB, (uint64_t)BH * m, SB) &&
         make_map_strided(&P.tmARs, dtype, w.aR, SB, (uint64_t)BH * m, SB) &&
         make_map_strided(&P.tmOut, dtype, Y, SB, (uint64_t)BH * m, SB);
  }
  if (!ok) return 7;
  P.aL = (uint8_t*)w.aL; P.aR = (uint8_t*)w.aR; P.y = (uint8_t*)w.y; P.out = (uint8_t*)Y;
  P.cL = w.cL; P.cR = w.cR; P.status = w.status; P.counters = counters;
  P.trace = trace_buffer();
  P.m = m; P.BH = BH; P.T = T_steps; P.H = H; P.lse = lse; P.n_valid = n_valid;
  P.tiles_per_head = m / (kRows / SB);
  P.tiles_per_phase = BH * P.tiles_per_head;
  P.scale = scale;
  P.n_counters = 2 * T_steps * BH;
  P.wait_cycles = knobs().wait_cycles;
  if (!ws_armed) {   // status block and counters start at zero; the kernel leaves them that way
    if (cudaMemsetAsync(ws, 0, kWsStatusBytes, st) != cudaSuccess) return 7;
    if (cudaMemsetAsync(counters, 0, counters_bytes(BH, T_steps), st) != cudaSuccess) return 7;
  }
  static int num_sms = 0;
  if (num_sms == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 7;
  }
  const void* fn = (const void*)monarch_persistent<T, B, SB>;
  if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) != cudaSuccess)
    return 7;
  const int total = 2 * T_steps * P.tiles_per_phase;
  int n = 0;
  if (mode == 0 || mode == 2) {   // one launch, dependencies tracked by counters
    P.g_begin = knobs().skip_first_half_step ? P.tiles_per_phase : 0; P.g_end = total; P.check_deps = 1;
    const int grid = total < num_sms ? total : num_sms;
    if (mode == 0) {
      if (launch_decoupled<T, B, SB>(P, grid, st) != cudaSuccess) return 7;
    } else {
      monarch_persistent<T, B, SB><<<grid, kThreads, kSmem, st>>>(P);
    }
    n = 1;
  } else {                  // one launch per half-step (stream order is the dependency)
    P.check_deps = 0;
    for (int p = 0; p < 2 * T_steps; ++p) {
      P.g_begin = p * P.tiles_per_phase; P.g_end = P.g_begin + P.tiles_per_phase;
      const int grid = P.tiles_per_phase < num_sms ? P.tiles_per_phase : num_sms;
      monarch_persistent<T, B, SB><<<grid, kThreads, kSmem, st>>>(P);
      ++n;
    }
  }
  if (cudaGetLastError() != cudaSuccess) return 7;
  *launches = n;
  return 0;
}

inline int launch(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int b, int T,
                  int dtype, float scale, void* ws, cudaStream_t st, int* launches, int mode,
                  bool ws_armed, int H = 0, float* lse = nullptr, int n_valid = 0) {
#define MA_TP_ARGS Q, K, V, Y, BH, N, T, dtype, scale, ws, st, launches, mode, ws_armed, H, lse, n_valid
  if (dtype == 1) {
    if (b == 128) return launch_t<__half, 128, 128>(MA_TP_ARGS);
    if (b == 64) return launch_t<__half, 64, 64>(MA_TP_ARGS);
    return launch_t<__half, 64, 32>(MA_TP_ARGS);
  }
  if (b == 128) return launch_t<__nv_bfloat16, 128, 128>(MA_TP_ARGS);
  if (b == 64) return launch_t<__nv_bfloat16, 64, 64>(MA_TP_ARGS);
  return launch_t<__nv_bfloat16, 64, 32>(MA_TP_ARGS);
#undef MA_TP_ARGS
}

}  // namespace tp
}  // namespace ma
