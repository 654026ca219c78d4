// Persistent tensor-core kernel with the softmax weights handed to the apply MMA through tensor
// memory (MA_PATH_TENSOR_TMEM): f16/bf16, d = 64, m = b in {64, 128}.
//
// Tiles, order, dependency counters and the MMAs' mathematics are those described in
// tensor_persistent.cuh and tensor_path.cuh.  What this kernel changes is where a tile's data live
// while it is in flight, because the tile rate is set by how long a tile holds each resource
// (tensor-memory columns, operand slots) along its chain
// (load -> score MMA -> softmax -> apply MMA -> epilogue -> store):
//   * a softmax thread reads its whole score row into registers at once and gives the score stage
//     back before it computes anything: two score stages suffice and nothing in tensor memory is held
//     during the softmax;
//   * R and final L half-steps: the 16-bit weights are written (tcgen05.st) to a small stage of
//     their own, one per softmax group, and the apply MMA takes them from there as its A operand.
//     No P buffer in shared memory, no shared-memory traffic for P in either direction;
//   * non-final L half-step (the apply MMA contracts over the ROW index of the weights, so it needs
//     them transposed, which only a shared-memory operand can be): the normalised weights go over
//     the tile's own alpha_L operand, dead once the score MMA has run, and (b = 128, two 64-column
//     chunks) over a slot of the V ring, idle in that half-step;
//   * the output accumulators are two units of 64 columns: a tile takes one (alpha_L, alpha_R or Y)
//     or two (alpha_L and y on the last R half-step, alpha_R and the c_R columns on a non-final L
//     half-step), each unit is handed to the epilogue and given back on its own;
//   * the shared memory this frees holds deeper operand rings and a second staging buffer;
//   * softmax warpgroups run with 200 registers (setmaxnreg; the other warps give theirs up).
// 512 threads: warp 0 TMA producer, warp 1 MMA issuer (both poll), warps 2-3 store threads (one per
// staging buffer), warps 4-7 and 8-11 softmax groups (alternate tiles), warps 12-15 epilogue group.
// TMEM (512 columns): score stages of B columns from column 0, the two weight stages of B / 2
// columns from column 256, the two output units from column 384.
#pragma once
#include <type_traits>

#include "tensor_persistent.cuh"

namespace ma {
namespace tp3 {

using namespace ma::tensor;
using ma::tp::Params;
using ma::tp::Tile;
using ma::tp::TileIter;
using ma::tp::stamp;
using ma::tp::mbar_arrive;
using ma::tp::ld_acquire;
using ma::tp::bulk_load_1d;
using ma::tp::tmem_ld1;
using ma::tp::tma_store_commit;
using ma::tp::tma_store_wait_read;
using ma::tp::tma_store_wait_all;

constexpr int kThreads = 512;
constexpr int kSlot = kTileBytes;

template <int B>
struct Cfg;
#ifndef MA_T3_E
#define MA_T3_E 4
#define MA_T3_L 5
#define MA_T3_V 2
#endif
template <>
struct Cfg<128> {
  static constexpr int kRingE = MA_T3_E, kRingL = MA_T3_L, kRingV = MA_T3_V, kStagesS = 2;
};
template <>
struct Cfg<64> {
  static constexpr int kRingE = 4, kRingL = 5, kRingV = 2, kStagesS = 4;
};
constexpr int kMaxRing = 6, kMaxStagesS = 4, kStatSlots = 8;
constexpr uint32_t kTmemP = 256, kTmemO = 384;   // first column of the weight stages / output units

template <int B>
struct Lay {
  using C = Cfg<B>;
  static constexpr int E = 0;
  static constexpr int L = E + C::kRingE * kSlot;
  static constexpr int V = L + C::kRingL * kSlot;
  static constexpr int Stage = V + C::kRingV * kSlot;   // two staging buffers
  static constexpr int Ones = Stage + 2 * kSlot;        // 2 KB
  static constexpr int Vec = Ones + 2048;               // kRingL x 128 floats (c_R / c_L)
  static constexpr int Stat = Vec + C::kRingL * 512;    // kStatSlots x 128 floats (1 / row sum)
  static constexpr int Bars = Stat + kStatSlots * 512;
  static constexpr int Total = Bars + 512;
  static constexpr int kSmem = Total + 1024;
  static_assert(kSmem <= 227 * 1024, "shared memory budget");
  static_assert(C::kStagesS * B <= (int)kTmemP && kTmemP + B <= kTmemO, "tensor memory budget");
};

struct __align__(8) Bars {
  uint64_t fullL[kMaxRing], emptyL[kMaxRing];   // fullL: all operands of a tile (E, L, c-vector)
  uint64_t emptyE[kMaxRing];
  uint64_t fullV[kMaxRing], emptyV[kMaxRing];
  uint64_t s_ready[kMaxStagesS], s_free[kMaxStagesS];
  uint64_t p_ready[2], p_free[2];               // weight stage of softmax group c
  uint64_t o_ready[2], o_free[2];               // output unit u
  uint64_t stage_ready[2], stage_free[2];
  uint32_t tmem_slot;
  volatile int abort_flag;
  long long wait_limit;
};
static_assert(sizeof(Bars) <= 512, "barrier block");

__device__ __forceinline__ uint32_t mbar_poll_addr(uint32_t addr, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(addr), "r"(parity)
      : "memory");
  return done;
}

template <int N>
struct RingPos {
  int slot = 0;
  uint32_t par = 0;
  __device__ __forceinline__ void advance() {
    if (++slot == N) { slot = 0; par ^= 1; }
  }
};

// Bounded wait: a wait that runs out records where in the status word and raises the CTA's abort
// flag; from then on every wait of the CTA returns at once, so all roles run through their
// remaining (now meaningless) tiles without blocking and the kernel ends.
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

// tcgen05.mma with the A operand in tensor memory (16-bit elements, two per 32-bit column, one
// row per lane: the layout of the accumulator the weights were computed from).
template <bool ACC>
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc,
                                        uint32_t idesc) {
  if (ACC)
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc)
        : "memory");
  else
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 0, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc)
        : "memory");
}

// D[row, :] = sum_c P[row, c] X[c, :] with P in tensor memory (columns tmem_p ...: 16-bit pairs)
// and X = [X0 | X1] read MN-major from [B rows][64] shared-memory tiles (N = 64 nb).
template <int B, int FT>
__device__ __forceinline__ void issue_apply_ts(uint32_t tmem_o, uint32_t tmem_p, uint32_t sX0,
                                               uint32_t x_chunk_stride, int nb) {
  const uint32_t idesc = instr_desc2(B, 64 * nb, FT, FT, 0, 1);
  const uint64_t dX = smem_desc(sX0, x_chunk_stride, 1024);
#pragma unroll
  for (int t = 0; t < Geo<B>::kTiles; ++t) {
    const uint32_t lane_off = (uint32_t)(t * 16) << 16;
#pragma unroll
    for (int ks = 0; ks < B / 16; ++ks) {
      const uint64_t db = dX + (uint64_t)((t * (B * 128) + ks * 2048) >> 4);
      if (ks == 0) umma_ts<false>(tmem_o + lane_off, tmem_p + lane_off + 8 * ks, db, idesc);
      else umma_ts<true>(tmem_o + lane_off, tmem_p + lane_off + 8 * ks, db, idesc);
    }
  }
}

// Non-final L half-step: D[c, 0:64] = sum_row P[row, c] X[row, :] at tmem_o and sixteen copies of
// sum_row P[row, c] at tmem_c.
// P is in shared memory, [64-column chunk][rows][128 bytes]; the chunks are `p_chunk_stride` bytes
// apart (they need not be adjacent).
template <int B, int FT>
__device__ __forceinline__ void issue_transposed_apply_split(uint32_t tmem_o, uint32_t tmem_c,
                                                             uint32_t sP, uint32_t p_chunk_stride,
                                                             uint32_t sX, uint32_t sOnes) {
  constexpr uint32_t idesc = instr_desc2(B, 64, FT, FT, 1, 1);
  constexpr uint32_t idesc1 = instr_desc2(B, 16, FT, FT, 1, 0);
  const uint64_t ones = smem_desc(sOnes, 16, 1024);
  const uint64_t dP = smem_desc(sP, p_chunk_stride, 1024);
  const uint64_t dX = smem_desc(sX, 16, 1024);
#pragma unroll
  for (int t = 0; t < Geo<B>::kTiles; ++t) {
    const uint32_t d = tmem_o + ((uint32_t)(t * 16) << 16);
    const uint32_t dc = tmem_c + ((uint32_t)(t * 16) << 16);
#pragma unroll
    for (int ks = 0; ks < B / 16; ++ks) {
      const uint64_t off = (uint64_t)((t * (B * 128) + ks * 2048) >> 4);
      if (ks == 0) {
        umma_c<false>(d, dP + off, dX + off, idesc);
        umma_c<false>(dc, dP + off, ones, idesc1);
      } else {
        umma_c<true>(d, dP + off, dX + off, idesc);
        umma_c<true>(dc, dP + off, ones, idesc1);
      }
    }
  }
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, "
      "%12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, "
      "%30, %31, %32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
      "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
      "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
      "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
template <int REGS>
__device__ __forceinline__ void reg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS));
}
template <int REGS>
__device__ __forceinline__ void reg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS));
}
// all bulk-store groups of this thread but the newest one are complete
__device__ __forceinline__ void tma_store_wait_all_but_one() {
  asm volatile("cp.async.bulk.wait_group 1;" ::: "memory");
}

// Eight 16-byte chunks (64 16-bit values, already packed in pairs) of row `srow` of a
// [rows][128 bytes] tile with 128-byte swizzled rows.
__device__ __forceinline__ void store_packed_row64(uint8_t* tile, int srow, const uint32_t* u) {
  uint8_t* base = tile + srow * 128;
#pragma unroll
  for (int c = 0; c < 8; ++c)
    *reinterpret_cast<uint4*>(base + ((c ^ (srow & 7)) << 4)) =
        make_uint4(u[4 * c], u[4 * c + 1], u[4 * c + 2], u[4 * c + 3]);
}

template <typename T, int B, bool TRACE>
__global__ void __launch_bounds__(kThreads, 1) monarch_tmem(const __grid_constant__ Params P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  using Lay = tp3::Lay<B>;
  using C = Cfg<B>;
  constexpr int kRingE = C::kRingE, kRingL = C::kRingL, kRingV = C::kRingV;
  constexpr int kStagesS = C::kStagesS;
  Bars* bars = reinterpret_cast<Bars*>(smem + Lay::Bars);
  constexpr int kBlocks = kRows / B;          // blocks (k of an R tile, j of an L tile) per CTA
  constexpr int FT = Fmt<T>::code;
  constexpr int NP = B / 2;                   // 32-bit columns of a row of 16-bit weights
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m = P.m;
  const int lastR = 2 * P.T - 2;

  if (tid == 0) {
    for (int i = 0; i < kRingL; ++i) { mbar_init(&bars->fullL[i], 1); mbar_init(&bars->emptyL[i], 1); }
    for (int i = 0; i < kRingE; ++i) mbar_init(&bars->emptyE[i], 1);
    for (int i = 0; i < kRingV; ++i) { mbar_init(&bars->fullV[i], 1); mbar_init(&bars->emptyV[i], 1); }
    for (int i = 0; i < kStagesS; ++i) { mbar_init(&bars->s_ready[i], 1); mbar_init(&bars->s_free[i], 128); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->p_ready[i], 128);
      mbar_init(&bars->p_free[i], 1);
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
    const uint32_t one2 = pack2<T>(1.f, 1.f);
    *reinterpret_cast<uint4*>(smem + Lay::Ones + tid * 16) = make_uint4(one2, one2, one2, one2);
  }
  if (warp == 0) tmem_alloc(&bars->tmem_slot, 512);

  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_slot;
  const uint32_t tmem_p = tmem + kTmemP;         // weight stage c at tmem_p + c * (B / 2)
  const uint32_t tmem_o = tmem + kTmemO;         // output unit u at tmem_o + 64 u

  const int first_g = P.g_begin + blockIdx.x;
  const int stride_g = gridDim.x;
  const int n_total = first_g < P.g_end ? (P.g_end - first_g + stride_g - 1) / stride_g : 0;
  // V ring: V tile (last R half-step), y tile (final L half-step), and at b = 128 the second
  // 64-column chunk of the weights of a non-final L half-step
  auto needs_v = [&](const Tile& t) { return t.isR ? t.withV : (t.final_ || B == 128); };
  // staging rounds of a tile: alpha_L (R) or alpha_R / Y (L); y on the last R half-step
  auto rounds_of = [&](const Tile& t) { return (t.isR && t.withV) ? 2 : 1; };
  // output units of a tile: one per staging round; a non-final L tile takes a second one for c_R
  auto units_of = [&](const Tile& t) { return ((t.isR && t.withV) || (!t.isR && !t.final_)) ? 2 : 1; };

  if (warp < 4) {
    reg_dec<48>();
    if (warp == 0) {
      // ---------------------------------------------------------------- TMA producer (polling)
      if (lane == 0) {
        const bool deps = P.check_deps != 0;
        auto counter_of = [&](const Tile& t) { return P.counters + (t.p - 1) * P.BH + t.h; };
        // rounds the half-step before t's stores per head
        auto need_of = [&](const Tile& t) { return P.tiles_per_head * ((t.p - 1) == lastR ? 2 : 1); };
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
            const Tile t = itE.get();
            bool ok = !deps || t.p == 0 || ctrE >= need_of(t);
            if (!ok) {
              ctrE = ld_acquire(counter_of(t));
              ok = ctrE >= need_of(t);
            }
            if (ok) {
              const int eE = rE.slot, eL = rL.slot;
              asm volatile("fence.proxy.async.global;" ::: "memory");
              uint8_t* sE = smem + Lay::E + eE * kSlot;
              uint8_t* sL = smem + Lay::L + eL * kSlot;
              const bool needC = !t.first;
              float* sC = reinterpret_cast<float*>(smem + Lay::Vec) + eL * 128;
              mbar_expect_tx(&bars->fullL[eL], 2 * kSlot + (needC ? 512 : 0));
              if (t.isR) {
                const int row0 = (t.h * m + t.idx0) * B;
                if (needC) bulk_load_1d(sC, P.cR + row0, 512, &bars->fullL[eL]);
                if (t.first) tma_load_2d(sE, &P.tmQ, &bars->fullL[eL], 0, row0);
                else tma_load_2d(sE, &P.tmAR, &bars->fullL[eL], 0, row0);
                tma_load_2d(sL, &P.tmK, &bars->fullL[eL], 0, row0);
              } else {
                const int row0 = (t.h * B + t.idx0) * m;
                bulk_load_1d(sC, P.cL + row0, 512, &bars->fullL[eL]);
                tma_load_2d(sE, &P.tmAL, &bars->fullL[eL], 0, row0);
                // one box: kBlocks blocks (positions j) of B rows (l) each, block after block
                tma_load_3d(sL, &P.tmQs, &bars->fullL[eL], 0, t.h * m, t.idx0);
              }
              if (TRACE) stamp(P, nE, 0);
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
            const Tile t = itV.get();
            bool ok = !deps || t.p == 0 || ctrV >= need_of(t);
            if (!ok) {
              ctrV = ld_acquire(counter_of(t));
              ok = ctrV >= need_of(t);
            }
            if (ok) {
              const int eV = rV.slot;
              if (!t.isR && !t.final_) {
                // the slot is lent to the tile's softmax group (second chunk of its weights)
                mbar_arrive(&bars->fullV[eV]);
              } else {
                asm volatile("fence.proxy.async.global;" ::: "memory");
                uint8_t* sV = smem + Lay::V + eV * kSlot;
                mbar_expect_tx(&bars->fullV[eV], kSlot);
                if (t.isR) tma_load_2d_hint(sV, &P.tmV, &bars->fullV[eV], 0, (t.h * m + t.idx0) * B, pol_first);
                else tma_load_2d(sV, &P.tmY, &bars->fullV[eV], 0, (t.h * B + t.idx0) * m);
              }
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
      // ---------------------------------------------------------------- MMA issuer (polling)
      // Two pending jobs are polled, never waited for: the apply MMA of the oldest unfinished tile
      // (needs the weights of its softmax group) and the score MMA of the next tile (needs its
      // operands, which may depend on other CTAs).  Blocking on the second would hold up the first
      // and could deadlock the grid.
      if (elect_one()) {
        const uint32_t sE0 = smem_u32(smem + Lay::E), sL0 = smem_u32(smem + Lay::L);
        const uint32_t sV0 = smem_u32(smem + Lay::V);
        const uint32_t sOnes = smem_u32(smem + Lay::Ones);
        int i1 = 0, i2 = 0;
        int uc = 0;                                 // output units handed out so far
        TileIter it1(P, first_g, stride_g, kBlocks), it2(P, first_g, stride_g, kBlocks);
        long long t0 = 0;
        bool idle = false;
        RingPos<kRingE> r1E, r2E;
        RingPos<kRingL> r1L, r2L;
        RingPos<kStagesS> r1S;
        RingPos<kRingV> rV;
        RingPos<2> r2P;                             // weight stage (softmax group) of tile i2
        uint32_t p_par = 0;
        const uint32_t bFullL = smem_u32(&bars->fullL[0]), bSFree = smem_u32(&bars->s_free[0]);
        const uint32_t bFullV = smem_u32(&bars->fullV[0]), bPReady = smem_u32(&bars->p_ready[0]);
        const uint32_t bOFree = smem_u32(&bars->o_free[0]);
        while (i2 < n_total) {
          bool did = false;
          const int c = r2P.slot;
          const int uA = uc & 1, uB = uA ^ 1;
          const uint32_t r_ready = mbar_poll_addr(bPReady + c * 8, p_par);
          const uint32_t r_ofA = mbar_poll_addr(bOFree + uA * 8, ((uc >> 1) & 1) ^ 1);
          const uint32_t r_ofB = mbar_poll_addr(bOFree + uB * 8, (((uc + 1) >> 1) & 1) ^ 1);
          const uint32_t r_v = mbar_poll_addr(bFullV + rV.slot * 8, rV.par);
          const uint32_t r_l = mbar_poll_addr(bFullL + r1L.slot * 8, r1L.par);
          const uint32_t r_sf = mbar_poll_addr(bSFree + r1S.slot * 8, r1S.par ^ 1);
          if (i2 < i1 && (r_ready & r_ofA)) {
            const Tile t = it2.get();
            const bool needV = needs_v(t);
            const int nu = units_of(t);
            if ((!needV || r_v) && (nu == 1 || r_ofB)) {
              const int eL2 = r2L.slot, eV = rV.slot, eE2 = r2E.slot;
              const uint32_t sL = sL0 + eL2 * kSlot, sV = sV0 + eV * kSlot, sE = sE0 + eE2 * kSlot;
              const uint32_t tOA = tmem_o + 64 * uA, tOB = tmem_o + 64 * uB, tP = tmem_p + c * NP;
              tc_fence_after();
              if (t.isR) {
                issue_apply_ts<B, FT>(tOA, tP, sL, 16, 1);               // alpha_L = P K
                umma_commit(&bars->o_ready[uA]);
                if (needV) {
                  issue_apply_ts<B, FT>(tOB, tP, sV, 16, 1);             // y = P V
                  umma_commit(&bars->o_ready[uB]);
                }
                umma_commit(&bars->emptyL[eL2]);
                umma_commit(&bars->p_free[c]);
              } else if (t.final_) {
                issue_apply_ts<B, FT>(tOA, tP, sV, 16, 1);               // Y = P y
                umma_commit(&bars->o_ready[uA]);
                umma_commit(&bars->emptyL[eL2]);
                umma_commit(&bars->p_free[c]);
              } else {
                // weights: chunk 0 over the tile's alpha_L operand, chunk 1 (b = 128) in the V slot;
                // alpha_R into unit A, the c_R columns into unit B
                issue_transposed_apply_split<B, FT>(tOA, tOB, sE, B == 128 ? (sV - sE) : kSlot, sL, sOnes);
                umma_commit(&bars->o_ready[uA]);
                umma_commit(&bars->o_ready[uB]);
                umma_commit(&bars->emptyE[eE2]);
                umma_commit(&bars->emptyL[eL2]);
                umma_commit(&bars->p_free[c]);             // (keeps the barrier's phase in step)
              }
              if (needV) { umma_commit(&bars->emptyV[eV]); rV.advance(); }
              if (TRACE) stamp(P, i2, 4);
              ++i2;
              it2.next();
              r2L.advance();
              r2E.advance();
              r2P.advance();
              if (r2P.slot == 0) p_par ^= 1;
              uc += nu;
              did = true;
            }
          }
          if (i1 < n_total && (r_l & r_sf)) {
            const Tile t = it1.get();
            const int eE = r1E.slot, eL1 = r1L.slot, s1 = r1S.slot;
            tc_fence_after();
            const uint32_t sE = sE0 + eE * kSlot, sL = sL0 + eL1 * kSlot;
            // R: A = aR (E ring), B = K (L ring).  L: A = Qb (L ring), B = aL (E ring).
            issue_scores<B, FT>(tmem + s1 * B, t.isR ? sE : sL, t.isR ? sL : sE);
            // (a non-final L tile keeps its E slot for its weights until the apply MMA has run)
            if (t.isR || t.final_) umma_commit(&bars->emptyE[eE]);
            umma_commit(&bars->s_ready[s1]);
            if (TRACE) stamp(P, i1, 1);
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
    } else {
      // ---------------------------------------------------------------- store threads
      // Thread w owns staging buffer w, i.e. the staging rounds r = w, w + 2, ...  A round's store
      // is complete (its rows readable by other CTAs) some time after the buffer has been read; the
      // thread bumps the tile's dependency counter then.  If the next round is already staged it
      // does not wait for that but issues the next store first (two stores in flight per thread);
      // otherwise it waits at once, so that no counter is ever held back by work that may depend on
      // it.
      if (lane == 0) {
        const int w = warp - 2;
        const uint8_t* sStage = smem + Lay::Stage + w * kSlot;
        const uint64_t pol_first = policy_evict_first();
        TileIter it(P, first_g, stride_g, kBlocks);
        int round = 0, mine = 0;                 // staging rounds so far: all, and this thread's
        int* pending = nullptr;                  // counter of a store not yet known complete
        // (a reduction with release semantics: nothing comes back, so the thread does not wait for
        // the round trip to the counter's home in L2 as it would with a fence and an atomic)
        auto signal = [&](int* ctr) {
          asm volatile("fence.proxy.async.global;" ::: "memory");
          asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(ctr) : "memory");
        };
        for (int n = 0; n < n_total; ++n, it.next()) {
          const Tile t = it.get();
          const int nr = rounds_of(t);
          for (int r = 0; r < nr; ++r, ++round) {
            if ((round & 1) != w) continue;
            wait_or_abort(&bars->stage_ready[w], mine & 1, bars, P.status, 40);
            // one box per round: the tile's kBlocks blocks of B rows (blocked views)
            if (t.isR) tma_store_3d(r == 0 ? &P.tmALs : &P.tmYs, sStage, 0, t.h * B, t.idx0);
            else if (t.final_) tma_store_3d_hint(&P.tmOut, sStage, 0, t.h * m, t.idx0, pol_first);
            else tma_store_3d(&P.tmARs, sStage, 0, t.h * m, t.idx0);
            tma_store_commit();
            if (pending != nullptr) {
              tma_store_wait_all_but_one();
              signal(pending);
            }
            tma_store_wait_read();
            mbar_arrive(&bars->stage_free[w]);
            pending = P.counters + t.p * P.BH + t.h;
            ++mine;
            if (!mbar_poll_addr(smem_u32(&bars->stage_ready[w]), mine & 1)) {
              tma_store_wait_all();
              signal(pending);
              pending = nullptr;
            }
          }
        }
        if (pending != nullptr) {
          tma_store_wait_all();
          signal(pending);
        }
      }
    }
  } else if (warp < 12) {
    // ------------------------------------------------------------------ softmax groups
    reg_inc<200>();
    const int c = (warp - 4) >> 2;             // group; takes tiles n = c, c + 2, ...
    const int sub = warp & 3;
    const int t_row = sub * 32 + lane;         // TMEM lane = score row owned by this thread
    const int tile = Geo<B>::tile(t_row), r = Geo<B>::row(t_row), srow = tile * B + r;
    float* stat = reinterpret_cast<float*>(smem + Lay::Stat);
    const bool stamper = (sub == 0 && lane == 0);

    TileIter it(P, first_g, stride_g, kBlocks);
    int nV = 0;                                // V-ring allocations before tile n
    for (int n = 0; n < n_total; ++n, it.next()) {
      const Tile t = it.get();
      const bool usesV = needs_v(t);
      const int eV = nV % kRingV;
      const uint32_t parV = (nV / kRingV) & 1;
      if (usesV) ++nV;
      if ((n & 1) != c) continue;
      const int eL = n % kRingL, eE = n % kRingE, s = n % kStagesS;
      const float* cv = reinterpret_cast<const float*>(smem + Lay::Vec) + eL * 128;
      const uint32_t tS = tmem + s * B + ((uint32_t)(sub * 32) << 16);
      wait_or_abort(&bars->s_ready[s], (n / kStagesS) & 1, bars, P.status, 30);
      tc_fence_after();
      if (TRACE && stamper) stamp(P, n, 2);
      // the state tile the score MMA consumed is read exactly once: drop its lines from L2
      if (t.isR) {
        if (!t.first) discard_line(P.aR + ((size_t)(t.h * m + t.idx0) * B + t_row) * 128);
      } else {
        discard_line(P.aL + ((size_t)(t.h * B + t.idx0) * m + t_row) * 128);
      }

      float x[B];
#pragma unroll
      for (int cc = 0; cc < B / 32; ++cc) tmem_ld32(tS + 32 * cc, x + 32 * cc);
      tmem_ld_wait();
      tc_fence_before();
      mbar_arrive(&bars->s_free[s]);           // the row is in registers: the stage may be reused
      const uint32_t tP = tmem_p + c * NP + ((uint32_t)(sub * 32) << 16);
      const uint32_t parP = ((n >> 1) & 1) ^ 1;   // the apply MMA of this group's previous tile is done
      uint32_t u[NP];
      float inv_s;
      if (t.isR) {
        // Z_R = scale * S / c_R (Eq. 7); c_L = sum R log R (Eq. 10)
        float inv_c = 1.f;
        if (!t.first) {
          const float cr = cv[srow];
          inv_c = cr > 1e-30f ? 1.f / cr : 0.f;
        }
        const float f = P.scale * inv_c * kLog2e;
        float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < B / 2; ++i) m4[i & 3] = max3(m4[i & 3], x[2 * i], x[2 * i + 1]);
        const float mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        const float2 f2 = make_float2(f, f), off2 = make_float2(-mx * f, -mx * f);
        float2 a2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
        float2 z2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
        for (int i = 0; i < B / 2; ++i) {
          const float2 xv = make_float2(x[2 * i], x[2 * i + 1]);
          const float2 zz = ffma2(xv, f2, off2);
          const float2 pp = make_float2(fast_exp2(zz.x), fast_exp2(zz.y));
          z2[i & 1] = ffma2(pp, xv, z2[i & 1]);
          a2[i & 1] = fadd2(a2[i & 1], pp);
          u[i] = pack2<T>(pp.x, pp.y);
        }
        const float sum = (a2[0].x + a2[0].y) + (a2[1].x + a2[1].y);
        const float sz = (z2[0].x + z2[0].y) + (z2[1].x + z2[1].y);
        inv_s = 1.f / sum;
        wait_or_abort(&bars->p_free[c], parP, bars, P.status, 33);
        tc_fence_after();
#pragma unroll
        for (int cc = 0; cc < NP / 32; ++cc) tmem_st32(tP + 32 * cc, u + 32 * cc);
        // -c_L in log2 units, ready to be the addend of the next L half-step's logits
        P.cL[((size_t)t.h * B + r) * m + t.idx0 + tile] = fast_log2(sum) - f * (sz * inv_s - mx);
        tmem_st_wait();
      } else {
        // Z_L = scale * S' - c_L (Eq. 8), softmax over k = along the row
        const float f = P.scale * kLog2e;
        const float2 f2 = make_float2(f, f);
        const float4* cv4 = reinterpret_cast<const float4*>(cv + tile * B);
        float m4[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < B / 4; ++i) {
          const float4 k4 = cv4[i];
          const float2 za = ffma2(make_float2(x[4 * i], x[4 * i + 1]), f2, make_float2(k4.x, k4.y));
          const float2 zb = ffma2(make_float2(x[4 * i + 2], x[4 * i + 3]), f2, make_float2(k4.z, k4.w));
          m4[0] = max3(m4[0], za.x, za.y);
          m4[1] = max3(m4[1], zb.x, zb.y);
          x[4 * i] = za.x;
          x[4 * i + 1] = za.y;
          x[4 * i + 2] = zb.x;
          x[4 * i + 3] = zb.y;
        }
        const float mx = fmaxf(m4[0], m4[1]);
        const float2 nmx2 = make_float2(-mx, -mx);
        float2 a2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
        for (int i = 0; i < B / 2; ++i) {
          const float2 zz = fadd2(make_float2(x[2 * i], x[2 * i + 1]), nmx2);
          const float2 pp = make_float2(fast_exp2(zz.x), fast_exp2(zz.y));
          a2[i & 1] = fadd2(a2[i & 1], pp);
          x[2 * i] = pp.x;
          x[2 * i + 1] = pp.y;
        }
        const float sum = (a2[0].x + a2[0].y) + (a2[1].x + a2[1].y);
        inv_s = 1.f / sum;
        if (t.final_) {
          // the apply MMA contracts over k: weights unnormalised, the epilogue divides
#pragma unroll
          for (int i = 0; i < B / 2; ++i) u[i] = pack2<T>(x[2 * i], x[2 * i + 1]);
          wait_or_abort(&bars->p_free[c], parP, bars, P.status, 33);
          tc_fence_after();
#pragma unroll
          for (int cc = 0; cc < NP / 32; ++cc) tmem_st32(tP + 32 * cc, u + 32 * cc);
          tmem_st_wait();
        } else {
          // the apply MMA contracts over rows: weights normalised in fp32, rounded once, written to
          // shared memory over the alpha_L operand the score MMA is done with (and the lent V slot)
          const float2 is2 = make_float2(inv_s, inv_s);
#pragma unroll
          for (int i = 0; i < B / 2; ++i) {
            const float2 v = fmul2(make_float2(x[2 * i], x[2 * i + 1]), is2);
            u[i] = pack2<T>(v.x, v.y);
          }
          // (the weights do not use the group's stage in tensor memory, but its "ready" barrier
          // must not complete a second phase before the MMA issuer has seen the first)
          wait_or_abort(&bars->p_free[c], parP, bars, P.status, 33);
          store_packed_row64(smem + Lay::E + eE * kSlot, srow, u);
          if (B == 128) {
            wait_or_abort(&bars->fullV[eV], parV, bars, P.status, 34);
            store_packed_row64(smem + Lay::V + eV * kSlot, srow, u + (B == 128 ? 32 : 0));
          }
          fence_proxy_async();
        }
      }
      stat[(n & (kStatSlots - 1)) * 128 + t_row] = inv_s;     // for the epilogue group
      tc_fence_before();
      mbar_arrive(&bars->p_ready[c]);
      if (TRACE && stamper) stamp(P, n, 3);
    }
  } else {
    // ------------------------------------------------------------------ epilogue group: O -> rows
    reg_dec<64>();
    const int sub = warp & 3;
    const int t_row = sub * 32 + lane;
    const int tile = Geo<B>::tile(t_row), r = Geo<B>::row(t_row), srow = tile * B + r;
    const float* stat = reinterpret_cast<const float*>(smem + Lay::Stat);
    const uint32_t tO0 = tmem_o + ((uint32_t)(sub * 32) << 16);
    const bool stamper = (sub == 0 && lane == 0);
    TileIter it(P, first_g, stride_g, kBlocks);
    int round = 0, uc = 0;                     // staging rounds / output units so far
    for (int n = 0; n < n_total; ++n, it.next()) {
      const Tile t = it.get();
      const int nr = rounds_of(t);
      const bool scaled = t.isR || t.final_;
      float c1 = 0.f, inv_s = 1.f;
      float buf[32];
      for (int rr = 0; rr < nr; ++rr, ++round, ++uc) {
        const int u = uc & 1;
        const uint32_t tO = tO0 + 64 * u;
        const int sb = round & 1;
        uint8_t* sStage = smem + Lay::Stage + sb * kSlot;
        wait_or_abort(&bars->stage_free[sb], ((round >> 1) & 1) ^ 1, bars, P.status, 35);
        wait_or_abort(&bars->o_ready[u], (uc >> 1) & 1, bars, P.status, 31);
        tc_fence_after();
        if (TRACE && stamper && rr == 0) stamp(P, n, 5);
        if (rr == 0) inv_s = stat[(n & (kStatSlots - 1)) * 128 + t_row];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          tmem_ld32(tO + 32 * half, buf);
          tmem_ld_wait();
          if (half == 1) {                       // the unit is in registers: give it back
            tc_fence_before();
            mbar_arrive(&bars->o_free[u]);
            if (TRACE && stamper && rr == nr - 1) stamp(P, n, 7);
          }
          if (scaled) store_row32<T>(sStage, srow, 32 * half, buf, inv_s);
          else store_row32<T>(sStage, srow, 32 * half, buf);
        }
        fence_proxy_async();
        mbar_arrive(&bars->stage_ready[sb]);
      }
      if (!scaled) {                             // c_R: first column of the second unit
        const int u = uc & 1;
        wait_or_abort(&bars->o_ready[u], (uc >> 1) & 1, bars, P.status, 32);
        tc_fence_after();
        c1 = tmem_ld1(tO0 + 64 * u);
        tmem_ld_wait();
        tc_fence_before();
        mbar_arrive(&bars->o_free[u]);
        ++uc;
      }
      if (t.final_) discard_line(P.y + ((size_t)(t.h * B + t.idx0) * m + t_row) * 128);
      if (!scaled) P.cR[((size_t)t.h * m + r) * B + t.idx0 + tile] = c1;
      if (TRACE && stamper) stamp(P, n, 6);
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
  if (tid == 0) {   // the last CTA re-arms the dependency counters
    __threadfence();
    if (atomicAdd(P.status + 1, 1) == (int)gridDim.x - 1) {
      for (int i = 0; i < P.n_counters; ++i) P.counters[i] = 0;
      P.status[1] = 0;
    }
  }
}

template <typename T, int B, bool TRACE>
inline cudaError_t launch_kernel_x(const Params& P, int grid, cudaStream_t st) {
  const void* fn = (const void*)monarch_tmem<T, B, TRACE>;
  constexpr int kSmem = Lay<B>::kSmem;
  static bool prepared[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!prepared[dev]) {
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    prepared[dev] = true;
  }
  monarch_tmem<T, B, TRACE><<<grid, kThreads, kSmem, st>>>(P);
  return cudaGetLastError();
}

}  // namespace tp3

namespace tp {
template <typename T, int B>
cudaError_t launch_tmem(const Params& P, int grid, cudaStream_t st) {
  if (P.trace != nullptr) return tp3::launch_kernel_x<T, B, true>(P, grid, st);
  return tp3::launch_kernel_x<T, B, false>(P, grid, st);
}
#ifdef MA_TU_TENSOR_TMEM
template cudaError_t launch_tmem<__half, 128>(const Params&, int, cudaStream_t);
template cudaError_t launch_tmem<__half, 64>(const Params&, int, cudaStream_t);
template cudaError_t launch_tmem<__nv_bfloat16, 128>(const Params&, int, cudaStream_t);
template cudaError_t launch_tmem<__nv_bfloat16, 64>(const Params&, int, cudaStream_t);
#endif
}  // namespace tp
}  // namespace ma
