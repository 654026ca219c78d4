// Persistent tensor-core kernel with P handed to the apply MMA through shared memory
// (MA_PATH_TENSOR): tiles, order and dependency counters as described in tensor_persistent.cuh.
//   * two softmax warpgroups do nothing but S -> P (alternate tiles); S has three (b = 128) or four
//     (b <= 64) TMEM stages, so the score MMA runs ahead and a group never waits for it;
//   * a third warpgroup does every epilogue (O -> 16-bit rows -> staging), so the softmax groups
//     never wait for the apply MMA; O has one TMEM stage at b = 128 and two at b <= 64;
//   * two store threads alternate tiles (TMA store, completion, dependency counter).
// 512 threads: warp 0 TMA producer, warp 1 MMA issuer, warps 2-3 store threads, warps 4-7 and
// 8-11 softmax groups, warps 12-15 epilogue group.  The producer and the MMA issuer poll: each
// iteration issues all its barrier tests back to back, then acts on whatever is ready.
// TMEM: score stages of B columns from column 0, then the O stages of 128 columns.  Shared memory
// (see Cfg / Lay): rings E / L / V of 16 KB operand tiles, one P buffer per softmax group, one
// 16 KB staging buffer (the last R half-step stages alpha_L and y in two rounds), row statistics,
// c-vectors, a tile of ones.
//
// bf16 with b = 32 (HILO): the 8-bit mantissa of alpha_L is the dominant error of a bf16 pipeline
// when the logits are large (it is multiplied by Q into logits of size ~100), and at this shape's
// logit scale it alone pushes some heads past 1e-2.  alpha_L is therefore stored as two bf16 arrays,
// hi = bf16(x) and lo = bf16(x - hi) (one more staging round in the R half-steps), the L half-steps
// load both tiles into a double-size E slot and the score MMA runs twice into the same stage; and the
// R half-step sums (and takes the entropy over) the weights as rounded to bf16, so that the rounding
// of a dominant weight cancels in alpha_L = sum(P K) / sum(P).
//
// Measured and rejected on B200 (slower than this arrangement): issuing the first half of the apply
// MMA while the softmax is still producing the second half of P (it holds the single O stage for
// half a softmax); writing rows to global memory straight from the epilogue threads instead of
// staging + TMA store (16-byte stores to rows 128 bytes apart swamp the load/store unit, the
// softmax groups slow down by half); one store thread instead of two (the completion fence of a tile
// is about a microsecond); separate blocking issuer threads for the two MMAs.
#pragma once
#include <type_traits>

#include "tensor_persistent.cuh"

namespace ma {
namespace tp2 {

using namespace ma::tensor;
using ma::tp::Params;
using ma::tp::Tile;
using ma::tp::TileIter;
using ma::tp::stamp;
using ma::tp::mbar_test;
using ma::tp::mbar_arrive;
using ma::tp::ld_acquire;
using ma::tp::bulk_load_1d;
using ma::tp::tmem_ld1;
using ma::tp::tma_store_commit;
using ma::tp::tma_store_wait_read;
using ma::tp::tma_store_wait_all;

constexpr int kThreads = 512;
constexpr int kSlot = kTileBytes;

// Pipeline depths per MMA block size.  TMEM has 512 columns: a score stage takes B of them, an O
// stage 128.  Shared memory: operand rings of 16 KB tiles, one P buffer per softmax group, one
// staging buffer.  The L ring is the deepest: its tile (K, or the Q block of an L half-step) is held
// from the load until the apply MMA of the tile has run, four to five microseconds.
// HILO (bf16 with b = 32): alpha_L travels as a hi + lo pair of 16-bit tiles, so an E slot holds
// two tiles (32 KB) and the rings are shallower.
template <int B, bool HILO>
struct Cfg;
template <>
struct Cfg<128, false> {
  static constexpr int kRingE = 2, kRingL = 4, kRingV = 2, kStagesS = 3, kStagesO = 1;
};
template <>
struct Cfg<64, false> {
  static constexpr int kRingE = 3, kRingL = 5, kRingV = 2, kStagesS = 4, kStagesO = 2;
};
template <>
struct Cfg<64, true> {
  static constexpr int kRingE = 2, kRingL = 4, kRingV = 2, kStagesS = 4, kStagesO = 2;
};
constexpr int kMaxRing = 6, kMaxStagesS = 4;

template <int B, bool HILO>
struct Lay {
  using C = Cfg<B, HILO>;
  static constexpr int kPBytes = 128 * B * 2;           // one P buffer (128 rows x B columns)
  static constexpr int kSlotE = HILO ? 2 * kSlot : kSlot;
  static constexpr int E = 0;
  static constexpr int L = E + C::kRingE * kSlotE;
  static constexpr int V = L + C::kRingL * kSlot;
  static constexpr int P = V + C::kRingV * kSlot;       // two P buffers
  static constexpr int Stage = P + 2 * kPBytes;         // 16 KB
  static constexpr int Ones = Stage + kSlot;            // 2 KB
  static constexpr int Vec = Ones + 2048;               // kRingL x 128 floats (c_R / c_L)
  static constexpr int Stat = Vec + C::kRingL * 512;    // 4 x 128 floats (1 / row sum)
  static constexpr int Bars = Stat + 4 * 512;
  static constexpr int Total = Bars + 512;
  static constexpr int kSmem = Total + 1024;
  static_assert(kSmem <= 227 * 1024, "shared memory budget");
  static_assert(C::kStagesS * B + C::kStagesO * 128 <= 512, "tensor memory budget");
};

struct __align__(8) Bars {
  uint64_t fullE[kMaxRing], emptyE[kMaxRing];
  uint64_t fullL[kMaxRing], emptyL[kMaxRing];
  uint64_t fullV[kMaxRing], emptyV[kMaxRing];
  uint64_t s_ready[kMaxStagesS];
  uint64_t p_ready[2], p_free[2];
  uint64_t o_ready[2], o_free[2], stage_ready[2], stage_free;
  uint32_t tmem_slot;
  volatile int abort_flag;
  long long wait_limit;
};
static_assert(sizeof(Bars) <= 512, "barrier block");

// Non-blocking phase test for the polling loops.  Shared memory is busy (MMA operand reads, TMA
// writes, P stores), so one barrier read takes a hundred cycles or more: a polling thread issues
// all its tests of an iteration back to back and only then looks at the results.
__device__ __forceinline__ uint32_t mbar_poll(uint64_t* bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(smem_u32(bar)), "r"(parity));
  return done;
}

// Position in a ring of N slots (or stages): slot index and the parity of the round, kept
// incrementally so that the polling threads do no divisions.
template <int N>
struct RingPos {
  int slot = 0;
  uint32_t par = 0;
  __device__ __forceinline__ void advance() {
    if (++slot == N) { slot = 0; par ^= 1; }
  }
};
__device__ __forceinline__ uint32_t mbar_poll_addr(uint32_t addr, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(addr), "r"(parity));
  return done;
}

// Bounded wait; see tensor_persistent.cuh (after a timeout every wait of the CTA returns at once).
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, Bars* bars, int* status,
                                              int where) {
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

// EXTRA: the rarely used hooks (inputs laid out [batch][N][heads][d], row log-sum-exp output, time
// stamps for the trace buffer) are
// compiled into a second instantiation: in the plain one they cost 4 % even when switched off (the
// producer's instruction stream is on the critical path and the compiler predicates the head
// index division instead of branching around it).
template <typename T, int B, int SB, bool EXTRA>
__global__ void __launch_bounds__(kThreads, 1) monarch_decoupled(const __grid_constant__ Params P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  constexpr bool HILO = std::is_same<T, __nv_bfloat16>::value && SB == 32;
  using Lay = tp2::Lay<B, HILO>;
  using C = Cfg<B, HILO>;
  constexpr int kSlotE = Lay::kSlotE;
  constexpr int kRingE = C::kRingE, kRingL = C::kRingL, kRingV = C::kRingV;
  constexpr int kStagesS = C::kStagesS, kStagesO = C::kStagesO;
  constexpr int kPBytes = Lay::kPBytes;
  Bars* bars = reinterpret_cast<Bars*>(smem + Lay::Bars);
  constexpr int kBlocks = kRows / SB;         // blocks (k of an R tile, j of an L tile) per CTA
  constexpr int NSUB = B / SB;                // blocks per MMA tile
  constexpr int FT = Fmt<T>::code;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m = P.m;

  if (tid == 0) {
    for (int i = 0; i < kRingE; ++i) { mbar_init(&bars->fullE[i], 1); mbar_init(&bars->emptyE[i], 1); }
    for (int i = 0; i < kRingL; ++i) { mbar_init(&bars->fullL[i], 1); mbar_init(&bars->emptyL[i], 1); }
    for (int i = 0; i < kRingV; ++i) { mbar_init(&bars->fullV[i], 1); mbar_init(&bars->emptyV[i], 1); }
    for (int i = 0; i < kStagesS; ++i) mbar_init(&bars->s_ready[i], 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->p_ready[i], 128);
      mbar_init(&bars->p_free[i], 1);
      mbar_init(&bars->o_ready[i], 1);
      mbar_init(&bars->o_free[i], 128);
    }
    mbar_init(&bars->stage_ready[0], 128);
    mbar_init(&bars->stage_ready[1], 128);
    mbar_init(&bars->stage_free, 1);
    bars->abort_flag = 0;
    bars->wait_limit = P.wait_cycles;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (tid < 128) {   // tile of ones for the column-sum MMA of the non-final L half-step
    const uint32_t one2 = pack2<T>(1.f, 1.f);
    *reinterpret_cast<uint4*>(smem + Lay::Ones + tid * 16) = make_uint4(one2, one2, one2, one2);
  }
  if (warp == 0) tmem_alloc(&bars->tmem_slot, 512);

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_slot;
  const uint32_t tmem_o = tmem + kStagesS * B;   // O stage o at tmem_o + 128 o

  const int first_g = P.g_begin + blockIdx.x;
  const int stride_g = gridDim.x;
  const int n_total = first_g < P.g_end ? (P.g_end - first_g + stride_g - 1) / stride_g : 0;
  auto needs_v = [&](const Tile& t) { return t.isR ? t.withV : t.final_; };
  // staging rounds of a tile: alpha_L (R) or alpha_R / Y (L), the low halves of alpha_L, y
  auto rounds_of = [&](const Tile& t) { return t.isR ? 1 + (HILO ? 1 : 0) + (t.withV ? 1 : 0) : 1; };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const bool deps = P.check_deps != 0;
      auto counter_of = [&](const Tile& t) { return P.counters + (t.p - 1) * P.BH + t.h; };
      int nE = 0, nVt = 0;
      TileIter itE(P, first_g, stride_g, kBlocks), itV(P, first_g, stride_g, kBlocks);
      while (nVt < n_total && !needs_v(itV.get())) { ++nVt; itV.next(); }
      const uint64_t pol_first = policy_evict_first();
      int ctrE = 0, ctrV = 0;
      if (deps && nE < n_total && itE.get().p > 0) ctrE = ld_acquire(counter_of(itE.get()));
      if (deps && nVt < n_total && itV.get().p > 0) ctrV = ld_acquire(counter_of(itV.get()));
      long long t0 = 0;
      bool idle = false;
      RingPos<kRingE> rE;
      RingPos<kRingL> rL;
      RingPos<kRingV> rV;
      const uint32_t bEmptyE = smem_u32(&bars->emptyE[0]), bEmptyL = smem_u32(&bars->emptyL[0]);
      const uint32_t bEmptyV = smem_u32(&bars->emptyV[0]);
      while (nE < n_total || nVt < n_total) {
        bool did = false;
        const uint32_t r_e = mbar_poll_addr(bEmptyE + rE.slot * 8, rE.par ^ 1);
        const uint32_t r_l = mbar_poll_addr(bEmptyL + rL.slot * 8, rL.par ^ 1);
        const uint32_t r_v = mbar_poll_addr(bEmptyV + rV.slot * 8, rV.par ^ 1);
        if (nE < n_total && (r_e & r_l)) {
          // (the prefetched counter is looked at only once the slots are free: by then its load
          // has long landed and the thread does not stall on it)
          bool ok = !deps || itE.p == 0 || ctrE >= P.tiles_per_head;
          if (!ok) {
            ctrE = ld_acquire(counter_of(itE.get()));
            ok = ctrE >= P.tiles_per_head;
          }
          if (ok) {
            const Tile t = itE.get();
            const int eE = rE.slot, eL = rL.slot;
            asm volatile("fence.proxy.async.global;" ::: "memory");
            uint8_t* sE = smem + Lay::E + eE * kSlotE;
            uint8_t* sL = smem + Lay::L + eL * kSlot;
            const bool needC = !t.first;
            float* sC = reinterpret_cast<float*>(smem + Lay::Vec) + eL * 128;
            // one "operands landed" barrier per tile (indexed like the L ring) for E, L and c
            mbar_expect_tx(&bars->fullL[eL],
                           ((HILO && !t.isR) ? 3 * kSlot : 2 * kSlot) + (needC ? 512 : 0));
            // inputs in [batch][N][heads][d]: column offset of the head, row index without it
            const int xin = (EXTRA && P.H) ? (t.h % P.H) * kD : 0, hin = (EXTRA && P.H) ? t.h / P.H : t.h;
            if (t.isR) {
              const int row0 = (t.h * m + t.idx0) * SB, row_in = (hin * m + t.idx0) * SB;
              if (needC) bulk_load_1d(sC, P.cR + row0, 512, &bars->fullL[eL]);
              if (t.first) tma_load_2d(sE, &P.tmQ, &bars->fullL[eL], xin, row_in);
              else tma_load_2d(sE, &P.tmAR, &bars->fullL[eL], 0, row0);
              tma_load_2d(sL, &P.tmK, &bars->fullL[eL], xin, row_in);
            } else {
              const int row0 = (t.h * SB + t.idx0) * m;
              bulk_load_1d(sC, P.cL + row0, 512, &bars->fullL[eL]);
              tma_load_2d(sE, &P.tmAL, &bars->fullL[eL], 0, row0);
              if (HILO) tma_load_2d(sE + kSlot, &P.tmALlo, &bars->fullL[eL], 0, row0);
              // one box: kBlocks blocks (positions j) of SB rows (l) each, block after block
              tma_load_3d(sL, &P.tmQs, &bars->fullL[eL], xin, hin * m, t.idx0);
            }
            if (EXTRA) stamp(P, nE, 0);
            ++nE;
            rE.advance();
            rL.advance();
            itE.next();
            // the next tile's counter is read now and looked at one iteration later
            if (deps && nE < n_total && itE.p > 0) ctrE = ld_acquire(counter_of(itE.get()));
            did = true;
          }
        }
        if (nVt < n_total && r_v) {
          bool ok = !deps || itV.p == 0 || ctrV >= P.tiles_per_head;
          if (!ok) {
            ctrV = ld_acquire(counter_of(itV.get()));
            ok = ctrV >= P.tiles_per_head;
          }
          if (ok) {
            const Tile t = itV.get();
            const int eV = rV.slot;
            asm volatile("fence.proxy.async.global;" ::: "memory");
            uint8_t* sV = smem + Lay::V + eV * kSlot;
            mbar_expect_tx(&bars->fullV[eV], kSlot);
            const int xin = (EXTRA && P.H) ? (t.h % P.H) * kD : 0, hin = (EXTRA && P.H) ? t.h / P.H : t.h;
            if (t.isR) tma_load_2d_hint(sV, &P.tmV, &bars->fullV[eV], xin, (hin * m + t.idx0) * SB, pol_first);
            else tma_load_2d(sV, &P.tmY, &bars->fullV[eV], 0, (t.h * SB + t.idx0) * m);
            rV.advance();
            do { ++nVt; itV.next(); } while (nVt < n_total && !needs_v(itV.get()));
            if (deps && nVt < n_total && itV.p > 0) ctrV = ld_acquire(counter_of(itV.get()));
            did = true;
          }
        }
        if (did) {
          idle = false;
        } else {
          if (!idle) {
            idle = true;
            t0 = clock64();
          } else if (bars->abort_flag) {
            break;   // stop issuing: what is in flight drains before the CTA leaves
          } else if (clock64() - t0 > P.wait_cycles) {
            report_timeout(P.status, 10);
            bars->abort_flag = 1;
            break;   // stop issuing: what is in flight drains before the CTA leaves
          }
          __nanosleep(32);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (polling)
    if (elect_one()) {
      const uint32_t sE0 = smem_u32(smem + Lay::E), sL0 = smem_u32(smem + Lay::L);
      const uint32_t sV0 = smem_u32(smem + Lay::V), sP0 = smem_u32(smem + Lay::P);
      const uint32_t sOnes = smem_u32(smem + Lay::Ones);
      int i1 = 0, i2 = 0;
      TileIter it1(P, first_g, stride_g, kBlocks), it2(P, first_g, stride_g, kBlocks);
      long long t0 = 0;
      bool idle = false;
      RingPos<kRingE> r1E;                        // score MMA: tile i1
      RingPos<kRingL> r1L, r2L;                   // apply MMA: tile i2
      RingPos<kStagesS> r1S;
      RingPos<kRingV> rV;
      RingPos<kStagesO> r2O;
      RingPos<2> r2P;                             // P buffer of tile i2 is i2 & 1; parity of i2 >> 1
      uint32_t p_par = 0;
      const uint32_t bFullL = smem_u32(&bars->fullL[0]);
      const uint32_t bFullV = smem_u32(&bars->fullV[0]), bPReady = smem_u32(&bars->p_ready[0]);
      const uint32_t bOFree = smem_u32(&bars->o_free[0]);
      while (i2 < n_total) {
        bool did = false;
        const int c = r2P.slot;
        const uint32_t r_ready = mbar_poll_addr(bPReady + c * 8, p_par);
        const uint32_t r_of = mbar_poll_addr(bOFree + r2O.slot * 8, r2O.par ^ 1);
        const uint32_t r_v = mbar_poll_addr(bFullV + rV.slot * 8, rV.par);
        const uint32_t r_l = mbar_poll_addr(bFullL + r1L.slot * 8, r1L.par);
        if (i2 < i1 && (r_ready & r_of)) {
          const Tile t = it2.get();
          const bool needV = needs_v(t);
          if (!needV || r_v) {
            const int eL2 = r2L.slot, eV = rV.slot, o2 = r2O.slot;
            const uint32_t sL = sL0 + eL2 * kSlot, sV = sV0 + eV * kSlot, sP = sP0 + c * kPBytes;
            const uint32_t tO = tmem_o + o2 * 128;
            tc_fence_after();
            if (t.isR) issue_apply<B, FT, 0>(tO, sP, sL, needV ? (sV - sL) : 16, needV ? 2 : 1);
            else if (t.final_) issue_apply<B, FT, 0>(tO, sP, sV, 16, 1);
            else issue_transposed_apply<B, FT>(tO, sP, sL, sOnes);
            umma_commit(&bars->emptyL[eL2]);
            if (needV) { umma_commit(&bars->emptyV[eV]); rV.advance(); }
            umma_commit(&bars->p_free[c]);
            umma_commit(&bars->o_ready[o2]);
            if (EXTRA) stamp(P, i2, 4);
            ++i2;
            it2.next();
            r2L.advance();
            r2O.advance();
            r2P.advance();
            if (r2P.slot == 0) p_par ^= 1;
            did = true;
          }
        }
        if (i1 < n_total && i1 < i2 + kStagesS && r_l) {
          const Tile t = it1.get();
          const int eE = r1E.slot, eL1 = r1L.slot, s1 = r1S.slot;
          tc_fence_after();
          const uint32_t sE = sE0 + eE * kSlotE, sL = sL0 + eL1 * kSlot;
          // R: A = aR (E ring), B = K (L ring).  L: A = Qb (L ring), B = aL (E ring).
          issue_scores<B, FT>(tmem + s1 * B, t.isR ? sE : sL, t.isR ? sL : sE);
          if (HILO && !t.isR) issue_scores<B, FT, FT, true>(tmem + s1 * B, sL, sE + kSlot);
          umma_commit(&bars->emptyE[eE]);
          umma_commit(&bars->s_ready[s1]);
          if (EXTRA) stamp(P, i1, 1);
          ++i1;
          it1.next();
          r1E.advance();
          r1L.advance();
          r1S.advance();
          did = true;
        }
        if (did) {
          idle = false;
        } else {
          if (!idle) {
            idle = true;
            t0 = clock64();
          } else if (bars->abort_flag) {
            break;   // stop issuing: what is in flight drains before the CTA leaves
          } else if (clock64() - t0 > P.wait_cycles) {
            report_timeout(P.status, 20);
            bars->abort_flag = 1;
            break;   // stop issuing: what is in flight drains before the CTA leaves
          }
          __nanosleep(20);
        }
      }
    }
  } else if (warp < 4) {
    // ------------------------------------------------------------------ store threads
    // Thread w handles the tiles n = w, w + 2, ... and has a "staged" barrier of its own, so that
    // each waiter is never more than one phase away from the barrier it waits on.
    if (lane == 0) {
      const int w = warp - 2;
      const uint8_t* sStage = smem + Lay::Stage;
      const uint64_t pol_first = policy_evict_first();
      TileIter it(P, first_g, stride_g, kBlocks);
      int round = 0;                           // staging rounds this thread has taken so far
      for (int n = 0; n < n_total; ++n, it.next()) {
        const Tile t = it.get();
        const int nr = rounds_of(t);
        if ((n & 1) == w) {
          for (int r = 0; r < nr; ++r) {
            wait_or_abort(&bars->stage_ready[w], (round + r) & 1, bars, P.status, 40);
            // one box per round: the tile's kBlocks blocks of SB rows (blocked views)
            if (t.isR) {
              tma_store_3d(r == 0 ? &P.tmALs : ((HILO && r == 1) ? &P.tmALlos : &P.tmYs), sStage, 0,
                           t.h * SB, t.idx0);
            } else if (t.final_) {
              tma_store_3d_hint(&P.tmOut, sStage, (EXTRA && P.H) ? (t.h % P.H) * kD : 0,
                                ((EXTRA && P.H) ? t.h / P.H : t.h) * m, t.idx0, pol_first);
            } else {
              tma_store_3d(&P.tmARs, sStage, 0, t.h * m, t.idx0);
            }
            tma_store_commit();
            tma_store_wait_read();
            mbar_arrive(&bars->stage_free);
          }
          tma_store_wait_all();                 // rows (and c_L / c_R) are in global memory
          // (a reduction with release semantics: nothing comes back, so the thread does not wait
          // for the round trip to the counter's home in L2 as it would with a fence and an atomic)
          asm volatile("fence.proxy.async.global;" ::: "memory");
          asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(P.counters + t.p * P.BH + t.h) : "memory");
          if (EXTRA) stamp(P, n, 7);
          round += nr;
        }
      }
    }
  } else if (warp < 12) {
    // ------------------------------------------------------------------ softmax groups: S -> P
    const int c = (warp - 4) >> 2;             // group = P buffer; takes tiles n = c, c + 2, ...
    const int sub = warp & 3;
    const int t_row = sub * 32 + lane;         // TMEM lane = score row owned by this thread
    const int tile = Geo<B>::tile(t_row), r = Geo<B>::row(t_row), srow = tile * B + r;
    const int sb = r / SB, rb = r - sb * SB;
    const int blk = tile * NSUB + sb;
    uint8_t* sP = smem + Lay::P + c * kPBytes;
    float* stat = reinterpret_cast<float*>(smem + Lay::Stat);
    const bool stamper = (sub == 0 && lane == 0);
    constexpr int NC = B / 32;
    auto mine = [&](int cc) { return SB == B || (32 * cc) / SB == sb; };

    TileIter it(P, first_g + c * stride_g, 2 * stride_g, kBlocks);
    for (int n = c; n < n_total; n += 2, it.next()) {
      const Tile t = it.get();
      const int q = n >> 1, eL = n % kRingL, s = n % kStagesS;
      const float* cv = reinterpret_cast<const float*>(smem + Lay::Vec) + eL * 128;
      const uint32_t tS = tmem + s * B + ((uint32_t)(sub * 32) << 16);
      wait_or_abort(&bars->s_ready[s], (n / kStagesS) & 1, bars, P.status, 30);
      tc_fence_after();
      if (EXTRA && stamper) stamp(P, n, 2);
      // the state tile MMA 1 consumed is read exactly once: drop its lines from L2
      if (t.isR) {
        if (!t.first) discard_line(P.aR + ((size_t)(t.h * m + t.idx0) * SB + t_row) * 128);
      } else {
        discard_line(P.aL + ((size_t)(t.h * SB + t.idx0) * m + t_row) * 128);
      }

      float buf[32];
      float f, inv_s, mx, sum, sz = 0.f;
      float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      float2 a2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      const float* cvt = cv + blk * SB;
      if (t.isR) {
        // Z_R = scale * S / c_R (Eq. 7); c_L = sum R log R (Eq. 10)
        float inv_c = 1.f;
        if (!t.first) {
          const float cr = cv[srow];
          inv_c = cr > 1e-30f ? 1.f / cr : 0.f;
        }
        f = P.scale * inv_c * kLog2e;
        float2 z2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
        // Padding mask (App. C.3): in the last key block the columns from `lim` on are keys past
        // n_valid; they take no part in the maximum and get weight 0.
        int lim = B;
        if (EXTRA && SB == B && P.n_valid != 0 && t.idx0 + blk == m - 1) lim = P.n_valid - (m - 1) * SB;
        if constexpr (SB == B) {
          // Every row owns all B columns: 16-column chunks, the load of the next chunk in flight
          // while the current one is worked on (TMEM reads compete with the MMAs' accumulator
          // traffic and are the longest stall of this pass).  Measured: 2 % on the whole call; the
          // same change in the L half-steps costs registers (spills) and loses more than it gains.
          constexpr int NC16 = B / 16;
          float* b0 = buf;
          float* b1 = buf + 16;
          tmem_ld16(tS, b0);
#pragma unroll
          for (int cc = 0; cc < NC16; ++cc) {
            float* cur = (cc & 1) ? b1 : b0;
            float* nxt = (cc & 1) ? b0 : b1;
            tmem_ld_wait();
            tmem_ld16(tS + 16 * ((cc + 1) % NC16), nxt);     // wraps to the first chunk of pass 2
            if (EXTRA && lim < B) {
#pragma unroll
              for (int i = 0; i < 16; ++i)
                if (16 * cc + i >= lim) cur[i] = -INFINITY;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) m4[i & 3] = max3(m4[i & 3], cur[2 * i], cur[2 * i + 1]);
          }
          mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
          const float2 f2 = make_float2(f, f), off2 = make_float2(-mx * f, -mx * f);
          // the apply MMA of this group's previous tile must be done with the P buffer
          wait_or_abort(&bars->p_free[c], (q & 1) ^ 1, bars, P.status, 33);
#pragma unroll
          for (int cc = 0; cc < NC16; ++cc) {
            float* cur = (cc & 1) ? b1 : b0;
            float* nxt = (cc & 1) ? b0 : b1;
            tmem_ld_wait();
            if (cc + 1 < NC16) tmem_ld16(tS + 16 * (cc + 1), nxt);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              float2 x = make_float2(cur[2 * i], cur[2 * i + 1]);
              if (EXTRA && lim < B) {      // masked keys: score 0 (any finite value), weight 0 below
                if (16 * cc + 2 * i >= lim) x.x = 0.f;
                if (16 * cc + 2 * i + 1 >= lim) x.y = 0.f;
              }
              const float2 zz = ffma2(x, f2, off2);
              float2 pp = exp2_pair(zz, i);
              if (EXTRA && lim < B) {
                if (16 * cc + 2 * i >= lim) pp.x = 0.f;
                if (16 * cc + 2 * i + 1 >= lim) pp.y = 0.f;
              }
              z2[i & 1] = ffma2(pp, x, z2[i & 1]);
              a2[i & 1] = fadd2(a2[i & 1], pp);
              cur[2 * i] = pp.x;
              cur[2 * i + 1] = pp.y;
            }
            store_row16<T>(sP, srow, 16 * cc, cur);
          }
        } else {
#pragma unroll
        for (int cc = 0; cc < NC; ++cc) {
          if (!mine(cc)) continue;
          tmem_ld32(tS + 32 * cc, buf);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) m4[i & 3] = max3(m4[i & 3], buf[2 * i], buf[2 * i + 1]);
        }
        mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        const float2 f2 = make_float2(f, f), off2 = make_float2(-mx * f, -mx * f);
        // the apply MMA of this group's previous tile must be done with the P buffer
        wait_or_abort(&bars->p_free[c], (q & 1) ^ 1, bars, P.status, 33);
#pragma unroll
        for (int cc = 0; cc < NC; ++cc) {
          float* sv = buf;
          if (mine(cc)) {
            tmem_ld32(tS + 32 * cc, buf);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float2 x = make_float2(sv[2 * i], sv[2 * i + 1]);
              const float2 zz = ffma2(x, f2, off2);
              float2 pp = exp2_pair(zz, i);
              // HILO: sums and entropy are taken over the weights as MMA 2 will see them (16-bit),
              // so that the rounding of a dominant weight cancels in alpha_L = sum(P K) / sum(P)
              if (HILO) pp = unpack2<T>(pack2<T>(pp.x, pp.y));
              z2[i & 1] = ffma2(pp, x, z2[i & 1]);
              a2[i & 1] = fadd2(a2[i & 1], pp);
              sv[2 * i] = pp.x;
              sv[2 * i + 1] = pp.y;
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) sv[i] = 0.f;
          }
          store_row32<T>(sP, srow, 32 * cc, sv);
        }
        }
        sum = (a2[0].x + a2[0].y) + (a2[1].x + a2[1].y);
        sz = (z2[0].x + z2[0].y) + (z2[1].x + z2[1].y);
        inv_s = 1.f / sum;
        // -c_L in log2 units, ready to be the addend of the next L half-step's logits
        P.cL[((size_t)t.h * SB + rb) * m + t.idx0 + blk] = fast_log2(sum) - f * (sz * inv_s - mx);
      } else {
        // Z_L = scale * S' - c_L (Eq. 8), softmax over k = along the row
        f = P.scale * kLog2e;
        const float2 f2 = make_float2(f, f);
        if constexpr (SB == B) {
          // Pass 1 forms the logits z = f s + c, takes their maximum and writes them back over s in
          // TMEM, so that pass 2 is the same loop as in the R half-step (no second read of the
          // c-vector, no second multiply-add); 16-column chunks, next load in flight.
          constexpr int NC16 = B / 16;
          float* b0 = buf;
          float* b1 = buf + 16;
          tmem_ld16(tS, b0);
#pragma unroll
          for (int cc = 0; cc < NC16; ++cc) {
            float* cur = (cc & 1) ? b1 : b0;
            float* nxt = (cc & 1) ? b0 : b1;
            tmem_ld_wait();
            if (cc + 1 < NC16) tmem_ld16(tS + 16 * (cc + 1), nxt);
            const float4* cv4 = reinterpret_cast<const float4*>(cvt + 16 * cc);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float4 k4 = cv4[i];
              const float2 za = ffma2(make_float2(cur[4 * i], cur[4 * i + 1]), f2, make_float2(k4.x, k4.y));
              const float2 zb = ffma2(make_float2(cur[4 * i + 2], cur[4 * i + 3]), f2, make_float2(k4.z, k4.w));
              m4[0] = max3(m4[0], za.x, za.y);
              m4[1] = max3(m4[1], zb.x, zb.y);
              cur[4 * i] = za.x;
              cur[4 * i + 1] = za.y;
              cur[4 * i + 2] = zb.x;
              cur[4 * i + 3] = zb.y;
            }
            tmem_st16(tS + 16 * cc, cur);
          }
          tmem_st_wait();                        // the logits are in TMEM before they are read back
          mx = fmaxf(m4[0], m4[1]);
          const float2 nmx2 = make_float2(-mx, -mx);
          // final: the weights go to the P buffer as they are formed (normalised in the epilogue);
          // non-final: they go back to TMEM and a third pass writes them normalised
          if (t.final_) wait_or_abort(&bars->p_free[c], (q & 1) ^ 1, bars, P.status, 33);
          tmem_ld16(tS, b0);
#pragma unroll
          for (int cc = 0; cc < NC16; ++cc) {
            float* cur = (cc & 1) ? b1 : b0;
            float* nxt = (cc & 1) ? b0 : b1;
            tmem_ld_wait();
            if (cc + 1 < NC16) tmem_ld16(tS + 16 * (cc + 1), nxt);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float2 zz = fadd2(make_float2(cur[2 * i], cur[2 * i + 1]), nmx2);
              const float2 pp = exp2_pair(zz, i);
              a2[i & 1] = fadd2(a2[i & 1], pp);
              cur[2 * i] = pp.x;
              cur[2 * i + 1] = pp.y;
            }
            if (t.final_) store_row16<T>(sP, srow, 16 * cc, cur);
            else tmem_st16(tS + 16 * cc, cur);
          }
          if (!t.final_) {
            // MMA 2 of this half-step contracts over rows, so P must be normalised before it is
            // read: third pass, fp32 weights from TMEM times 1 / sum, one rounding to 16 bits.
            tmem_st_wait();
            const float is_ = 1.f / ((a2[0].x + a2[0].y) + (a2[1].x + a2[1].y));
            const float2 is2 = make_float2(is_, is_);
            wait_or_abort(&bars->p_free[c], (q & 1) ^ 1, bars, P.status, 33);
            tmem_ld16(tS, b0);
#pragma unroll
            for (int cc = 0; cc < NC16; ++cc) {
              float* cur = (cc & 1) ? b1 : b0;
              float* nxt = (cc & 1) ? b0 : b1;
              tmem_ld_wait();
              if (cc + 1 < NC16) tmem_ld16(tS + 16 * (cc + 1), nxt);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const float2 v = fmul2(make_float2(cur[2 * i], cur[2 * i + 1]), is2);
                cur[2 * i] = v.x;
                cur[2 * i + 1] = v.y;
              }
              store_row16<T>(sP, srow, 16 * cc, cur);
            }
          }
        } else {
#pragma unroll
        for (int cc = 0; cc < NC; ++cc) {
          if (!mine(cc)) continue;
          tmem_ld32(tS + 32 * cc, buf);
          tmem_ld_wait();
          const float4* cv4 = reinterpret_cast<const float4*>(cvt + 32 * cc - sb * SB);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float4 k4 = cv4[i];
            const float2 za = ffma2(make_float2(buf[4 * i], buf[4 * i + 1]), f2, make_float2(k4.x, k4.y));
            const float2 zb = ffma2(make_float2(buf[4 * i + 2], buf[4 * i + 3]), f2, make_float2(k4.z, k4.w));
            m4[0] = max3(m4[0], za.x, za.y);
            m4[1] = max3(m4[1], zb.x, zb.y);
          }
        }
        mx = fmaxf(m4[0], m4[1]);
        const float2 nmx2 = make_float2(-mx, -mx);
        wait_or_abort(&bars->p_free[c], (q & 1) ^ 1, bars, P.status, 33);
#pragma unroll
        for (int cc = 0; cc < NC; ++cc) {
          float* sv = buf;
          if (mine(cc)) {
            tmem_ld32(tS + 32 * cc, buf);
            tmem_ld_wait();
            const float4* cv4 = reinterpret_cast<const float4*>(cvt + 32 * cc - sb * SB);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float4 k4 = cv4[i];
              float2 za = ffma2(make_float2(sv[4 * i], sv[4 * i + 1]), f2, make_float2(k4.x, k4.y));
              float2 zb = ffma2(make_float2(sv[4 * i + 2], sv[4 * i + 3]), f2, make_float2(k4.z, k4.w));
              za = fadd2(za, nmx2);
              zb = fadd2(zb, nmx2);
              const float2 pa = exp2_pair(za, 2 * i);
              const float2 pb = exp2_pair(zb, 2 * i + 1);
              a2[0] = fadd2(a2[0], pa);
              a2[1] = fadd2(a2[1], pb);
              sv[4 * i] = pa.x;
              sv[4 * i + 1] = pa.y;
              sv[4 * i + 2] = pb.x;
              sv[4 * i + 3] = pb.y;
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) sv[i] = 0.f;
          }
          store_row32<T>(sP, srow, 32 * cc, sv);
        }
        }
        sum = (a2[0].x + a2[0].y) + (a2[1].x + a2[1].y);
        inv_s = 1.f / sum;
        // Row b l + j (l = rb, j = idx0 + blk) of the final L half-step: its log-sum-exp; summed over
        // the rows of a head it is the value of the objective (Eq. 6) at the returned matrix.
        if (EXTRA && t.final_ && P.lse != nullptr)
          P.lse[(size_t)t.h * (SB * m) + (size_t)rb * SB + t.idx0 + blk] = (mx + fast_log2(sum)) * kLn2;
        if (!t.final_ && SB != B) {
          // MMA 2 of this half-step contracts over rows: P must be normalised before it is read.
          // The thread re-reads its own row, rescales in fp32, writes it back.
          const float2 is2 = make_float2(inv_s, inv_s);
#pragma unroll
          for (int c8 = 0; c8 < B / 8; ++c8) {
            uint4* ptr = reinterpret_cast<uint4*>(sP + (c8 >> 3) * kTileBytes + srow * 128 +
                                                  (((c8 & 7) ^ (srow & 7)) << 4));
            uint4 qv = *ptr;
            uint32_t* qp = reinterpret_cast<uint32_t*>(&qv);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 v = fmul2(unpack2<T>(qp[e]), is2);
              qp[e] = pack2<T>(v.x, v.y);
            }
            *ptr = qv;
          }
        }
      }
      stat[(n & 3) * 128 + t_row] = inv_s;     // for the epilogue group
      fence_proxy_async();
      tc_fence_before();
      mbar_arrive(&bars->p_ready[c]);
      if (EXTRA && stamper) stamp(P, n, 3);
    }
  } else {
    // ------------------------------------------------------------------ epilogue group: O -> rows
    const int sub = warp & 3;
    const int t_row = sub * 32 + lane;
    const int tile = Geo<B>::tile(t_row), r = Geo<B>::row(t_row), srow = tile * B + r;
    const int sb = r / SB, rb = r - sb * SB;
    const int blk = tile * NSUB + sb;
    uint8_t* sStage = smem + Lay::Stage;
    const float* stat = reinterpret_cast<const float*>(smem + Lay::Stat);
    const uint32_t tO0 = tmem_o + ((uint32_t)(sub * 32) << 16);
    const bool stamper = (sub == 0 && lane == 0);
    TileIter it(P, first_g, stride_g, kBlocks);
    int round = 0;
    for (int n = 0; n < n_total; ++n, it.next()) {
      const Tile t = it.get();
      const int o = n % kStagesO;
      const uint32_t tO = tO0 + o * 128;
      wait_or_abort(&bars->o_ready[o], (n / kStagesO) & 1, bars, P.status, 31);
      tc_fence_after();
      if (EXTRA && stamper) stamp(P, n, 5);
      const float inv_s = stat[(n & 3) * 128 + t_row];
      if (t.final_) discard_line(P.y + ((size_t)(t.h * SB + t.idx0) * m + t_row) * 128);
      const int nr = rounds_of(t);
      const bool scaled = t.isR || t.final_;
      float c1 = 0.f;
      if (!scaled) c1 = tmem_ld1(tO + 64);
      float buf[2][32];
      for (int rr = 0; rr < nr; ++rr) {
        // what this round stages: 0 = the rows (columns 0-63 of O), 1 = low halves of the same
        // values (alpha_L as a hi + lo pair), 2 = y (columns 64-127)
        const int kind = (t.isR && rr > 0) ? ((HILO && rr == 1) ? 1 : 2) : 0;
        if (kind != 1) {
          const int col = kind == 2 ? 64 : 0;
          tmem_ld32(tO + col, buf[0]);
          tmem_ld32(tO + col + 32, buf[1]);
          tmem_ld_wait();
        }
        if (rr == nr - 1) {                      // O is in registers: the next apply MMA may run
          tc_fence_before();
          mbar_arrive(&bars->o_free[o]);
        }
        wait_or_abort(&bars->stage_free, ((round + rr) & 1) ^ 1, bars, P.status, 35);
        if (kind == 1) {
          store_row32_lo<T>(sStage, srow, 0, buf[0], inv_s);
          store_row32_lo<T>(sStage, srow, 32, buf[1], inv_s);
        } else if (scaled) {
          store_row32<T>(sStage, srow, 0, buf[0], inv_s);
          store_row32<T>(sStage, srow, 32, buf[1], inv_s);
        } else {
          store_row32<T>(sStage, srow, 0, buf[0]);
          store_row32<T>(sStage, srow, 32, buf[1]);
        }
        fence_proxy_async();
        mbar_arrive(&bars->stage_ready[n & 1]);
      }
      if (!scaled) P.cR[((size_t)t.h * m + rb) * SB + t.idx0 + blk] = c1;
      if (EXTRA && stamper) stamp(P, n, 6);
      round += nr;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (bars->abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 200000) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 0) tmem_dealloc(tmem, 512);
  if (tid == 0) {   // the last CTA re-arms the dependency counters
    __threadfence();
    if (atomicAdd(P.status + 1, 1) == (int)gridDim.x - 1) {
      for (int i = 0; i < P.n_counters; ++i) P.counters[i] = 0;
      P.status[1] = 0;
    }
  }
}

template <typename T, int B, int SB, bool EXTRA>
inline cudaError_t launch_kernel_x(const Params& P, int grid, cudaStream_t st) {
  const void* fn = (const void*)monarch_decoupled<T, B, SB, EXTRA>;
  constexpr int kSmem = Lay<B, std::is_same<T, __nv_bfloat16>::value && SB == 32>::kSmem;
  cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
  if (e != cudaSuccess) return e;
  monarch_decoupled<T, B, SB, EXTRA><<<grid, kThreads, kSmem, st>>>(P);
  return cudaGetLastError();
}
template <typename T, int B, int SB>
inline cudaError_t launch_kernel(const Params& P, int grid, cudaStream_t st) {
  if (P.H != 0 || P.lse != nullptr || P.trace != nullptr || P.n_valid != 0)
    return launch_kernel_x<T, B, SB, true>(P, grid, st);
  return launch_kernel_x<T, B, SB, false>(P, grid, st);
}

}  // namespace tp2

namespace tp {
template <typename T, int B, int SB>
cudaError_t launch_decoupled(const Params& P, int grid, cudaStream_t st) {
  return tp2::launch_kernel<T, B, SB>(P, grid, st);
}
#ifdef MA_TU_TENSOR_DECOUPLED
template cudaError_t launch_decoupled<__half, 128, 128>(const Params&, int, cudaStream_t);
template cudaError_t launch_decoupled<__half, 64, 64>(const Params&, int, cudaStream_t);
template cudaError_t launch_decoupled<__half, 64, 32>(const Params&, int, cudaStream_t);
template cudaError_t launch_decoupled<__nv_bfloat16, 128, 128>(const Params&, int, cudaStream_t);
template cudaError_t launch_decoupled<__nv_bfloat16, 64, 64>(const Params&, int, cudaStream_t);
template cudaError_t launch_decoupled<__nv_bfloat16, 64, 32>(const Params&, int, cudaStream_t);
#endif
}  // namespace tp
}  // namespace ma
