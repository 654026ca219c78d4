// Tensor-core path of the MonarchAttention forward pass for sm_100a: TMA-fed tcgen05 MMAs with
// fp32 accumulators in tensor memory, 16-bit states in the workspace.
//
// Shapes: f16/bf16, d = 64, m = b in {64, 128}.  A CTA owns 128 score rows: one 128-row tile
// (b = 128) or two independent 64-row tiles (b = 64, placed in the lower and upper 16 lanes of every
// 32-lane TMEM sub-partition, so that all 128 threads own one row each).
//
//   R half-step, key block k (Eq. 7, 9 -> Eq. 10, and y of Eq. 4 on the last step):
//     S[j,i]  = aR_k[j,:] . K_k[i,:]                (MMA 1: A, B K-major from TMA tiles)
//     P       = exp(scale*S/cR[k,j] - rowmax)       (one thread per row, fp32, read from TMEM)
//     [aL|y]  = P [K_k | V_k] / rowsum              (MMA 2: A = P from smem, B = the same K tile
//                                                    read MN-major, V tile appended as N = 128)
//     cL[k,j] = sum_i R log R = (sum p z)/rowsum - rowmax - log rowsum
//   L half-step, in-block position j (Eq. 8, 10 -> Eq. 9, or the output of Eq. 4):
//     S'[l,k] = Qb_j[l,:] . aL_j[k,:]               (MMA 1; Qb_j rows fetched with stride b by TMA)
//     P'      = exp(scale*S' - cL[k,j] - rowmax)    (softmax over k = along the row)
//     not last: aR[k,:] = sum_l (P'/rowsum)[l,k] Qb_j[l,:]   (MMA 2 contracts over the ROW index:
//               A = P' read MN-major, B = Qb_j read MN-major), cR[k] = sum_l (P'/rowsum)[l,k]
//               (same A against a tile of ones)
//     last:     Y[b l + j,:] = P' y_j / rowsum      (MMA 2: A = P' K-major, B = y_j MN-major)
//
// The permutation P of the paper never moves data: it is the choice of TMA box strides when the
// states are stored (k-major tiles write j-major rows and vice versa).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace ma {
namespace tensor {

constexpr int kD = 64;              // head dimension handled by this path
constexpr int kRows = 128;          // score rows per CTA (= threads per CTA)
constexpr int kTileBytes = kRows * kD * 2;   // one [128][64] 16-bit tile, 128-byte swizzled rows
constexpr uint32_t kTmemCols = 256;
constexpr long long kWaitCycles = 2000000000LL;   // bound of every mbarrier wait (~1 s)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// ------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
// Bounded wait: returns false if the phase did not complete within kWaitCycles.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
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
    if (clock64() - t0 > kWaitCycles) return false;
  }
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, uint64_t* bar, int x,
                                            int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, "
      "%4}], [%2];" ::"r"(smem_u32(dst)),
      "l"((uint64_t)tm), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* tm, uint64_t* bar, int x,
                                            int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, "
      "%4, %5}], [%2];" ::"r"(smem_u32(dst)),
      "l"((uint64_t)tm), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}
// L2 eviction-priority policies for data that is touched once.
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_2d_hint(void* dst, const CUtensorMap* tm, uint64_t* bar,
                                                 int x, int y, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4}], [%2], %5;" ::"r"(smem_u32(dst)),
      "l"((uint64_t)tm), "r"(smem_u32(bar)), "r"(x), "r"(y), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_store_3d_hint(const CUtensorMap* tm, const void* src, int x,
                                                  int y, int z, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3, %4}], "
      "[%1], %5;" ::"l"((uint64_t)tm),
      "r"(smem_u32(src)), "r"(x), "r"(y), "r"(z), "l"(policy)
      : "memory");
}
// Drops a 128-byte line from L2 without writing it back (its contents become undefined).
__device__ __forceinline__ void discard_line(const void* p) {
  asm volatile("discard.global.L2 [%0], 128;" ::"l"(p) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* tm, const void* src, int x, int y,
                                             int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(
          (uint64_t)tm),
      "r"(smem_u32(src)), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void tma_store_commit_and_wait() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                   smem_u32(slot)),
               "r"(cols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                     uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Same with the accumulate flag known at compile time (no predicate register to set up).
template <bool ACC>
__device__ __forceinline__ void umma_c(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                       uint32_t idesc) {
  if (ACC)
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc)
        : "memory");
  else
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 0, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc)
        : "memory");
}
// One lane of a fully active warp (lets the compiler keep MMA operands in uniform registers).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   smem_u32(bar))
               : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, "
      "%12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, "
      "%30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, "
      "%12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
// Writes 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float* v) {
  const uint32_t* r = reinterpret_cast<const uint32_t*>(v);
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, "
      "%12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
      "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() {
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float fast_log2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ------------------------------------------------------------------------------------ descriptors
// Shared-memory matrix descriptor, 128-byte swizzle, sm_100 format: start address, leading byte
// offset (LBO) and stride byte offset (SBO) in 16-byte units, version 1, layout type 2.
//   K-major operand  ([MN rows][64 K elements] tile): SBO = 1024 B between 8-row groups, LBO unused.
//   MN-major operand ([K rows][64 MN elements] tile): SBO = 1024 B between 8-row (K) groups,
//                    LBO = distance between 64-element chunks along MN.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes,
                                              uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor of tcgen05.mma kind::f16: fp32 accumulate, A/B format (0 f16, 1 bf16),
// A/B major-ness (0 K-major, 1 MN-major), N >> 3, M >> 4.
__host__ __device__ constexpr uint32_t instr_desc2(int M, int N, int fmt_a, int fmt_b, int a_mn,
                                                   int b_mn) {
  return (1u << 4) | ((uint32_t)fmt_a << 7) | ((uint32_t)fmt_b << 10) | ((uint32_t)a_mn << 15) |
         ((uint32_t)b_mn << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, int fmt, int a_mn, int b_mn) {
  return instr_desc2(M, N, fmt, fmt, a_mn, b_mn);
}

template <typename T> struct Fmt;
template <> struct Fmt<__half> { static constexpr int code = 0; };
template <> struct Fmt<__nv_bfloat16> { static constexpr int code = 1; };

template <typename T> __device__ __forceinline__ uint32_t pack2(float a, float b);
template <> __device__ __forceinline__ uint32_t pack2<__half>(float a, float b) {
  __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
template <> __device__ __forceinline__ uint32_t pack2<__nv_bfloat16>(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

template <typename T> __device__ __forceinline__ float2 unpack2(uint32_t u);
template <> __device__ __forceinline__ float2 unpack2<__half>(uint32_t u) {
  return __half22float2(*reinterpret_cast<__half2*>(&u));
}
template <> __device__ __forceinline__ float2 unpack2<__nv_bfloat16>(uint32_t u) {
  return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
}

// Packed fp32 pairs (sm_100 f32x2 instructions: one issue slot for two lanes of work).
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
  float2 d;
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "mov.b64 rc, {%6, %7};\n\tfma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d.x), "=f"(d.y)
      : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
  return d;
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
  float2 d;
  asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "add.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d.x), "=f"(d.y)
      : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return d;
}
__device__ __forceinline__ float2 fmul2(float2 a, float2 b) {
  float2 d;
  asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "mul.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d.x), "=f"(d.y)
      : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return d;
}
// 2^x for a pair of non-positive arguments on the FMA and integer pipes (the special-function
// pipe, 16 results per clock per SM, is the busiest pipe of the softmax): round-to-nearest split
// x = n + r, |r| <= 1/2, cubic minimax polynomial for 2^r (max relative error 7.5e-5, well below
// 16-bit rounding), n added to the exponent field.  Arguments below -125 give ~2^-125.
__device__ __forceinline__ float2 exp2_poly2(float2 x) {
  x.x = fmaxf(x.x, -125.f);
  x.y = fmaxf(x.y, -125.f);
  const float2 magic = make_float2(12582912.f, 12582912.f);      // 1.5 * 2^23
  const float2 t = fadd2(x, magic);                               // low mantissa bits hold n
  const float2 n = fadd2(t, make_float2(-12582912.f, -12582912.f));
  const float2 r = ffma2(n, make_float2(-1.f, -1.f), x);
  float2 p = ffma2(r, make_float2(0.05517167f, 0.05517167f), make_float2(0.24261112f, 0.24261112f));
  p = ffma2(p, r, make_float2(0.69326099f, 0.69326099f));
  p = ffma2(p, r, make_float2(0.99992807f, 0.99992807f));
  p.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23));
  p.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23));
  return p;
}
// Pair i of a chunk: one pair in kPolyEvery takes the polynomial, the others ex2.approx
// (i is a compile-time constant after unrolling; 0 = never).  Alone on an SM the softmax pass is
// bound by the special-function pipe and one pair in four on the polynomial is the fastest mix;
// inside the persistent kernels it is bound by instruction issue (the pipe sits at 20 %), the
// polynomial's twelve instructions cost more than the two ex2 they replace, and "never" measured
// 4 % faster on the whole call at b = 128.
constexpr int kPolyEvery = 0;
__device__ __forceinline__ float2 exp2_pair(float2 z, int i) {
  if (kPolyEvery > 0 && i % (kPolyEvery > 0 ? kPolyEvery : 1) == kPolyEvery - 1) return exp2_poly2(z);
  return make_float2(fast_exp2(z.x), fast_exp2(z.y));
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Writes 32 consecutive columns [col0, col0+32) of row `srow` of a [chunks][128][64] 16-bit tile
// with 128-byte swizzled rows (the layout TMA produces and the MMA descriptors describe).
template <typename T>
__device__ __forceinline__ void store_row32(uint8_t* tile, int srow, int col0, const float* v,
                                            float mul) {
  uint8_t* base = tile + (col0 >> 6) * kTileBytes + srow * 128;
  const int c0 = (col0 & 63) >> 3;
  const float2 m2 = make_float2(mul, mul);
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const float2 a = fmul2(make_float2(v[8 * c + 0], v[8 * c + 1]), m2);
    const float2 b = fmul2(make_float2(v[8 * c + 2], v[8 * c + 3]), m2);
    const float2 cc = fmul2(make_float2(v[8 * c + 4], v[8 * c + 5]), m2);
    const float2 d = fmul2(make_float2(v[8 * c + 6], v[8 * c + 7]), m2);
    uint4 q;
    q.x = pack2<T>(a.x, a.y);
    q.y = pack2<T>(b.x, b.y);
    q.z = pack2<T>(cc.x, cc.y);
    q.w = pack2<T>(d.x, d.y);
    *reinterpret_cast<uint4*>(base + (((c0 + c) ^ (srow & 7)) << 4)) = q;
  }
}
// 16 consecutive columns, unscaled.
template <typename T>
__device__ __forceinline__ void store_row16(uint8_t* tile, int srow, int col0, const float* v) {
  uint8_t* base = tile + (col0 >> 6) * kTileBytes + srow * 128;
  const int c0 = (col0 & 63) >> 3;
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    uint4 q;
    q.x = pack2<T>(v[8 * c + 0], v[8 * c + 1]);
    q.y = pack2<T>(v[8 * c + 2], v[8 * c + 3]);
    q.z = pack2<T>(v[8 * c + 4], v[8 * c + 5]);
    q.w = pack2<T>(v[8 * c + 6], v[8 * c + 7]);
    *reinterpret_cast<uint4*>(base + (((c0 + c) ^ (srow & 7)) << 4)) = q;
  }
}
// The low halves of a hi + lo pair: what 16-bit rounding of v * mul dropped, rounded to 16 bits.
template <typename T>
__device__ __forceinline__ void store_row32_lo(uint8_t* tile, int srow, int col0, const float* v,
                                               float mul) {
  uint8_t* base = tile + (col0 >> 6) * kTileBytes + srow * 128;
  const int c0 = (col0 & 63) >> 3;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    uint32_t q[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float x0 = v[8 * c + 2 * e] * mul, x1 = v[8 * c + 2 * e + 1] * mul;
      const float2 hi = unpack2<T>(pack2<T>(x0, x1));
      q[e] = pack2<T>(x0 - hi.x, x1 - hi.y);
    }
    *reinterpret_cast<uint4*>(base + (((c0 + c) ^ (srow & 7)) << 4)) = make_uint4(q[0], q[1], q[2], q[3]);
  }
}
// Same without scaling.
template <typename T>
__device__ __forceinline__ void store_row32(uint8_t* tile, int srow, int col0, const float* v) {
  uint8_t* base = tile + (col0 >> 6) * kTileBytes + srow * 128;
  const int c0 = (col0 & 63) >> 3;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    uint4 q;
    q.x = pack2<T>(v[8 * c + 0], v[8 * c + 1]);
    q.y = pack2<T>(v[8 * c + 2], v[8 * c + 3]);
    q.z = pack2<T>(v[8 * c + 4], v[8 * c + 5]);
    q.w = pack2<T>(v[8 * c + 6], v[8 * c + 7]);
    *reinterpret_cast<uint4*>(base + (((c0 + c) ^ (srow & 7)) << 4)) = q;
  }
}

// ------------------------------------------------------------------------------------ shared state
struct __align__(8) Barriers {
  uint64_t load;
  uint64_t mma1;
  uint64_t mma2;
  uint32_t tmem_slot;
  uint32_t pad;
};

template <int B> struct Geo {
  static constexpr int kTiles = kRows / B;        // tiles per CTA
  static constexpr int kChunksP = B / 64;         // 64-column chunks of a P row
  // thread -> (tile, row in tile, smem row, TMEM lane offset of the tile)
  __device__ static __forceinline__ int tile(int t) { return B == 128 ? 0 : ((t & 31) >> 4); }
  __device__ static __forceinline__ int row(int t) {
    return B == 128 ? t : (((t >> 5) << 4) | (t & 15));
  }
};

// Issues MMA 1 (scores): both operands K-major [rows][64] tiles, K = d = 64 in four steps.
// FA / FB: element format of the A / B operand (0 f16, 1 bf16); the two may differ.
// ACC0: accumulate onto what the stage already holds (second half of a hi + lo operand pair).
template <int B, int FA, int FB = FA, bool ACC0 = false>
__device__ __forceinline__ void issue_scores(uint32_t tmem_s, uint32_t sA, uint32_t sB) {
  constexpr uint32_t idesc = instr_desc2(B, B, FA, FB, 0, 0);
#pragma unroll
  for (int t = 0; t < Geo<B>::kTiles; ++t) {
    const uint64_t da = smem_desc(sA + t * (B * 128), 16, 1024);
    const uint64_t db = smem_desc(sB + t * (B * 128), 16, 1024);
#pragma unroll
    for (int ks = 0; ks < kD / 16; ++ks) {
      if (ks == 0) umma_c<ACC0>(tmem_s + ((uint32_t)(t * 16) << 16), da, db, idesc);
      else umma_c<true>(tmem_s + ((uint32_t)(t * 16) << 16), da + 2 * ks, db + 2 * ks, idesc);
    }
  }
}

// Issues MMA 2 with A = P (K-major, [rows][B] in 64-column chunks) and B = [X0 | X1] read MN-major
// from [B rows][64] tiles (N = 64 * nb).  D[row, :] = sum_c P[row, c] X[c, :].
// PART: 0 = all k-steps, 1 = first half of the P columns only, 2 = second half only (so that the
// first half can run while the softmax is still producing the second).
template <int B, int FA, int PART = 0, int FB = FA>
__device__ __forceinline__ void issue_apply(uint32_t tmem_o, uint32_t sP, uint32_t sX0,
                                            uint32_t x_chunk_stride, int nb) {
  const uint32_t idesc = instr_desc2(B, 64 * nb, FA, FB, 0, 1);
  constexpr int KS = B / 16;
  constexpr int ks0 = PART == 2 ? KS / 2 : 0, ks1 = PART == 1 ? KS / 2 : KS;
  // One descriptor per operand; a k-step or tile only moves the start address (the field holds
  // address >> 4 and shared memory ends below 2^18, so adding to the low word cannot carry out).
  const uint64_t dP = smem_desc(sP, 16, 1024);
  const uint64_t dX = smem_desc(sX0, x_chunk_stride, 1024);
#pragma unroll
  for (int t = 0; t < Geo<B>::kTiles; ++t) {
#pragma unroll
    for (int ks = ks0; ks < ks1; ++ks) {
      const uint64_t da = dP + (uint64_t)(((ks >> 2) * kTileBytes + t * (B * 128) + (ks & 3) * 32) >> 4);
      const uint64_t db = dX + (uint64_t)((t * (B * 128) + ks * 2048) >> 4);
      if (ks == 0) umma_c<false>(tmem_o + ((uint32_t)(t * 16) << 16), da, db, idesc);
      else umma_c<true>(tmem_o + ((uint32_t)(t * 16) << 16), da, db, idesc);
    }
  }
}

// Issues MMA 2 of the non-final L half-step: contraction over the ROW index of P.
//   D[c, 0:64] = sum_row P[row, c] X[row, :],  D[c, 64:80] = sum_row P[row, c]  (tile of ones)
template <int B, int FA, int FB = FA>
__device__ __forceinline__ void issue_transposed_apply(uint32_t tmem_o, uint32_t sP, uint32_t sX,
                                                       uint32_t sOnes) {
  constexpr uint32_t idesc = instr_desc2(B, 64, FA, FB, 1, 1);
  constexpr uint32_t idesc1 = instr_desc2(B, 16, FA, FA, 1, 0);   // ones tile has A's format
  const uint64_t ones = smem_desc(sOnes, 16, 1024);
  const uint64_t dP = smem_desc(sP, kTileBytes, 1024);
  const uint64_t dX = smem_desc(sX, 16, 1024);
#pragma unroll
  for (int t = 0; t < Geo<B>::kTiles; ++t) {
    const uint32_t d = tmem_o + ((uint32_t)(t * 16) << 16);
#pragma unroll
    for (int ks = 0; ks < B / 16; ++ks) {
      const uint64_t off = (uint64_t)((t * (B * 128) + ks * 2048) >> 4);
      const uint64_t da = dP + off;
      const uint64_t db = dX + off;
      if (ks == 0) {
        umma_c<false>(d, da, db, idesc);
        umma_c<false>(d + 64, da, ones, idesc1);
      } else {
        umma_c<true>(d, da, db, idesc);
        umma_c<true>(d + 64, da, ones, idesc1);
      }
    }
  }
}

struct SmemLayout {
  // offsets from the 1024-byte aligned base
  static constexpr int A = 0;                         // aR tile / Qb tile; reused as staging
  static constexpr int X = kTileBytes;                // K tile / aL tile
  static constexpr int V = 2 * kTileBytes;            // V tile / y tile
  static constexpr int P = 3 * kTileBytes;            // P (up to two 64-column chunks)
  static constexpr int Ones = 5 * kTileBytes;         // 2 KB of 1.0
  static constexpr int Vec = Ones + 2048;             // 128 floats (cL column of the L step)
  static constexpr int Bars = Vec + 1024;
  static constexpr int Total = Bars + 64;
};
constexpr int kSmemBytes = SmemLayout::Total + 1024;  // slack for manual 1024-byte alignment

__device__ __forceinline__ void report_timeout(int* status, int where) {
  atomicCAS(status, 0, where);
}

// ------------------------------------------------------------------------------------ R half-step
// grid.x = BH * m / Geo<B>::kTiles; CTA c owns key blocks k0 .. k0 + kTiles - 1 of head h.
template <typename T, int B, bool FIRST, bool WITH_V>
__global__ void __launch_bounds__(kRows, 2)
r_step_tc(const __grid_constant__ CUtensorMap tmA,      // aR (or Q when FIRST): 2D [BH*N][64]
          const __grid_constant__ CUtensorMap tmK,      // K: 2D
          const __grid_constant__ CUtensorMap tmV,      // V: 2D
          const __grid_constant__ CUtensorMap tmAL,     // aL store: 3D (64, m, BH*b)
          const __grid_constant__ CUtensorMap tmYs,     // y store:  3D (64, m, BH*b)
          const float* __restrict__ cR, float* __restrict__ cL, int* status, int m, float scale) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  Barriers* bars = reinterpret_cast<Barriers*>(smem + SmemLayout::Bars);
  const int t = threadIdx.x, warp = t >> 5;
  constexpr int kTiles = Geo<B>::kTiles;
  constexpr int FMT = Fmt<T>::code;
  const int tiles_per_head = m / kTiles;
  const int h = blockIdx.x / tiles_per_head;
  const int k0 = (blockIdx.x - h * tiles_per_head) * kTiles;
  const int row0 = (h * m + k0) * B;          // first global row of this CTA's 128 rows

  if (t == 0) {
    mbar_init(&bars->load, 1);
    mbar_init(&bars->mma1, 1);
    mbar_init(&bars->mma2, 1);
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 0) tmem_alloc(&bars->tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_slot;
  const uint32_t tmem_s = tmem, tmem_o = tmem + B;

  if (t == 0) {
    mbar_expect_tx(&bars->load, (WITH_V ? 3 : 2) * kTileBytes);
    tma_load_2d(smem + SmemLayout::A, &tmA, &bars->load, 0, row0);
    tma_load_2d(smem + SmemLayout::X, &tmK, &bars->load, 0, row0);
    if (WITH_V) tma_load_2d(smem + SmemLayout::V, &tmV, &bars->load, 0, row0);
  }
  const int tile = Geo<B>::tile(t), r = Geo<B>::row(t), srow = tile * B + r;
  float inv_c = 1.f;
  if (!FIRST) {
    float c = cR[(size_t)row0 + srow];
    inv_c = c > 1e-30f ? 1.f / c : 0.f;
  }
  bool ok = true;
  if (t == 0) {
    ok = mbar_wait(&bars->load, 0);
    if (ok) {
      tc_fence_after();
      issue_scores<B, FMT>(tmem_s, smem_u32(smem + SmemLayout::A), smem_u32(smem + SmemLayout::X));
      umma_commit(&bars->mma1);
    } else {
      report_timeout(status, 1);
    }
  }
  if (__syncthreads_or(!ok)) goto cleanup;
  ok = mbar_wait(&bars->mma1, 0);
  if (!ok) report_timeout(status, 2);
  if (__syncthreads_or(!ok)) goto cleanup;
  tc_fence_after();
  {
    const uint32_t lane_addr = tmem_s + ((uint32_t)(warp * 32) << 16);
    float s[B];
#pragma unroll
    for (int c = 0; c < B / 32; ++c) tmem_ld32(lane_addr + 32 * c, s + 32 * c);
    tmem_ld_wait();
    const float f = scale * inv_c * kLog2e;
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < B; ++i) {
      s[i] *= f;
      mx = fmaxf(mx, s[i]);
    }
    float sum = 0.f, sz = 0.f;
#pragma unroll
    for (int i = 0; i < B; ++i) {
      const float p = fast_exp2(s[i] - mx);
      sz = fmaf(p, s[i], sz);
      sum += p;
      s[i] = p;
    }
#pragma unroll
    for (int c = 0; c < B / 32; ++c)
      store_row32<T>(smem + SmemLayout::P, srow, 32 * c, s + 32 * c);
    const float inv_s = 1.f / sum;
    cL[(size_t)row0 + srow] = kLn2 * (sz * inv_s - mx - fast_log2(sum));
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    if (t == 0) {
      tc_fence_after();
      issue_apply<B, FMT>(tmem_o, smem_u32(smem + SmemLayout::P), smem_u32(smem + SmemLayout::X),
                          SmemLayout::V - SmemLayout::X, WITH_V ? 2 : 1);
      umma_commit(&bars->mma2);
    }
    ok = mbar_wait(&bars->mma2, 0);
    if (!ok) report_timeout(status, 3);
    if (__syncthreads_or(!ok)) goto cleanup;
    tc_fence_after();
    // Epilogue: normalise, convert, stage (A tile for aL, P chunk 0 for y), TMA-store j-major.
    const uint32_t o_addr = tmem_o + ((uint32_t)(warp * 32) << 16);
#pragma unroll
    for (int half = 0; half < (WITH_V ? 2 : 1); ++half) {
      float o[64];
      tmem_ld32(o_addr + 64 * half, o);
      tmem_ld32(o_addr + 64 * half + 32, o + 32);
      tmem_ld_wait();
      uint8_t* stage = smem + (half == 0 ? SmemLayout::A : SmemLayout::P);
      store_row32<T>(stage, srow, 0, o, inv_s);
      store_row32<T>(stage, srow, 32, o + 32, inv_s);
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    if (t == 0) {
#pragma unroll
      for (int tt = 0; tt < kTiles; ++tt) {
        tma_store_3d(&tmAL, smem + SmemLayout::A + tt * (B * 128), 0, k0 + tt, h * B);
        if (WITH_V) tma_store_3d(&tmYs, smem + SmemLayout::P + tt * (B * 128), 0, k0 + tt, h * B);
      }
      tma_store_commit_and_wait();
    }
  }
cleanup:
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------------ L half-step
// grid.x = BH * b / Geo<B>::kTiles; CTA c owns in-block positions j0 .. j0 + kTiles - 1 of head h.
template <typename T, int B, bool FINAL>
__global__ void __launch_bounds__(kRows, 2)
l_step_tc(const __grid_constant__ CUtensorMap tmQs,     // Q strided view: 3D (64, b, BH*m)
          const __grid_constant__ CUtensorMap tmAL,     // aL: 2D [BH*b*m][64]
          const __grid_constant__ CUtensorMap tmY,      // y:  2D [BH*b*m][64]
          const __grid_constant__ CUtensorMap tmOut,    // aR (or Y when FINAL) strided view: 3D
          const float* __restrict__ cL, float* __restrict__ cR, int* status, int m, float scale) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  Barriers* bars = reinterpret_cast<Barriers*>(smem + SmemLayout::Bars);
  float* cvec = reinterpret_cast<float*>(smem + SmemLayout::Vec);   // [tile][k] : cL * log2e
  const int t = threadIdx.x, warp = t >> 5;
  constexpr int kTiles = Geo<B>::kTiles;
  constexpr int FMT = Fmt<T>::code;
  const int tiles_per_head = B / kTiles;      // b == m == B on this path
  const int h = blockIdx.x / tiles_per_head;
  const int j0 = (blockIdx.x - h * tiles_per_head) * kTiles;

  if (t == 0) {
    mbar_init(&bars->load, 1);
    mbar_init(&bars->mma1, 1);
    mbar_init(&bars->mma2, 1);
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 0) tmem_alloc(&bars->tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_slot;
  const uint32_t tmem_s = tmem, tmem_o = tmem + B;

  if (t == 0) {
    mbar_expect_tx(&bars->load, (FINAL ? 3 : 2) * kTileBytes);
#pragma unroll
    for (int tt = 0; tt < kTiles; ++tt)
      tma_load_3d(smem + SmemLayout::A + tt * (B * 128), &tmQs, &bars->load, 0, j0 + tt, h * m);
    tma_load_2d(smem + SmemLayout::X, &tmAL, &bars->load, 0, (h * B + j0) * m);
    if (FINAL) tma_load_2d(smem + SmemLayout::V, &tmY, &bars->load, 0, (h * B + j0) * m);
  }
  {
    // cL is stored [h][k][j]; this CTA needs column(s) j0 (+1): entry e = tile * B + k
    const int tile_e = t / B, k_e = t - tile_e * B;
    cvec[t] = cL[((size_t)h * m + k_e) * B + j0 + tile_e] * kLog2e;
    if (!FINAL) {
      // tile of ones for the column-sum MMA (2 KB = 1024 16-bit elements)
      uint32_t one2 = pack2<T>(1.f, 1.f);
      uint4 q = make_uint4(one2, one2, one2, one2);
      *reinterpret_cast<uint4*>(smem + SmemLayout::Ones + t * 16) = q;
    }
  }
  const int tile = Geo<B>::tile(t), r = Geo<B>::row(t), srow = tile * B + r;
  bool ok = true;
  if (t == 0) {
    ok = mbar_wait(&bars->load, 0);
    if (ok) {
      tc_fence_after();
      issue_scores<B, FMT>(tmem_s, smem_u32(smem + SmemLayout::A), smem_u32(smem + SmemLayout::X));
      umma_commit(&bars->mma1);
    } else {
      report_timeout(status, 4);
    }
  }
  if (__syncthreads_or(!ok)) goto cleanup;     // also publishes cvec and the ones tile
  ok = mbar_wait(&bars->mma1, 0);
  if (!ok) report_timeout(status, 5);
  if (__syncthreads_or(!ok)) goto cleanup;
  tc_fence_after();
  {
    const uint32_t lane_addr = tmem_s + ((uint32_t)(warp * 32) << 16);
    float s[B];
#pragma unroll
    for (int c = 0; c < B / 32; ++c) tmem_ld32(lane_addr + 32 * c, s + 32 * c);
    tmem_ld_wait();
    const float f = scale * kLog2e;
    const float* cv = cvec + tile * B;
    float mx = -INFINITY;
#pragma unroll
    for (int k = 0; k < B; ++k) {
      s[k] = fmaf(s[k], f, -cv[k]);
      mx = fmaxf(mx, s[k]);
    }
    float sum = 0.f;
#pragma unroll
    for (int k = 0; k < B; ++k) {
      s[k] = fast_exp2(s[k] - mx);
      sum += s[k];
    }
    const float inv_s = 1.f / sum;
    // not final: P is normalised before MMA 2 (the contraction runs over rows); final: afterwards
#pragma unroll
    for (int c = 0; c < B / 32; ++c)
      store_row32<T>(smem + SmemLayout::P, srow, 32 * c, s + 32 * c, FINAL ? 1.f : inv_s);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    if (t == 0) {
      tc_fence_after();
      if (FINAL)
        issue_apply<B, FMT>(tmem_o, smem_u32(smem + SmemLayout::P), smem_u32(smem + SmemLayout::V),
                            16, 1);
      else
        issue_transposed_apply<B, FMT>(tmem_o, smem_u32(smem + SmemLayout::P),
                                       smem_u32(smem + SmemLayout::A),
                                       smem_u32(smem + SmemLayout::Ones));
      umma_commit(&bars->mma2);
    }
    ok = mbar_wait(&bars->mma2, 0);
    if (!ok) report_timeout(status, 6);
    if (__syncthreads_or(!ok)) goto cleanup;
    tc_fence_after();
    // Epilogue.  FINAL: row = l, Y[b l + j] = D / rowsum.  Otherwise row = k: aR[k, j], cR[k, j].
    const uint32_t o_addr = tmem_o + ((uint32_t)(warp * 32) << 16);
    float o[64];
    tmem_ld32(o_addr, o);
    tmem_ld32(o_addr + 32, o + 32);
    if (!FINAL) {
      float c1[32];   // 16 identical column sums (and 16 unused columns)
      tmem_ld32(o_addr + 64, c1);
      tmem_ld_wait();
      cR[((size_t)h * m + r) * B + j0 + tile] = c1[0];
    } else {
      tmem_ld_wait();
    }
    uint8_t* stage = smem + SmemLayout::X;     // aL tile is dead after MMA 1
    store_row32<T>(stage, srow, 0, o, FINAL ? inv_s : 1.f);
    store_row32<T>(stage, srow, 32, o + 32, FINAL ? inv_s : 1.f);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    if (t == 0) {
#pragma unroll
      for (int tt = 0; tt < kTiles; ++tt)
        tma_store_3d(&tmOut, stage + tt * (B * 128), 0, j0 + tt, h * m);
      tma_store_commit_and_wait();
    }
  }
cleanup:
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------------ host side
constexpr size_t kWsStatusBytes = 256;

inline bool supported(int N, int d, int b, int m, int dtype, int BH) {
  if (dtype != 1 && dtype != 2) return false;
  if (d != kD || b != m) return false;
  if (b != 64 && b != 128) return false;
  if ((long long)BH * N >= (1LL << 31)) return false;
  return true;
}

struct Ws {
  int* status;
  void *aL, *aR, *y;
  float *cL, *cR;
  size_t bytes;
};
inline Ws ws_layout(void* base, int BH, int N) {
  Ws w;
  char* c = (char*)base;
  size_t off = 0;
  size_t big = ((size_t)BH * N * kD * 2 + 255) / 256 * 256;
  size_t small = ((size_t)BH * N * 4 + 255) / 256 * 256;
  w.status = (int*)(c + off); off += kWsStatusBytes;
  w.aL = c + off; off += big;
  w.aR = c + off; off += big;
  w.y = c + off; off += big;
  w.cL = (float*)(c + off); off += small;
  w.cR = (float*)(c + off); off += small;
  w.bytes = off;
  return w;
}
inline size_t workspace_bytes(int BH, int N, int d, int b, int T) {
  (void)d; (void)b; (void)T;
  return ws_layout(nullptr, BH, N).bytes;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) ==
            cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}
// 2D view [rows][64] of a contiguous 16-bit array, box = 128 rows.
inline bool make_map_rows(CUtensorMap* tm, int dtype, void* base, uint64_t rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {kD, rows};
  cuuint64_t strides[1] = {kD * 2};
  cuuint32_t box[2] = {kD, kRows};
  cuuint32_t es[2] = {1, 1};
  return fn(tm, dtype == 1 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
            base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// Row view of an input / output tensor.  H = 0: [batch*heads*N rows][64] as above, a tile is
// addressed (0, head * N + n).  H = heads: the tensor is [batch][N][heads][64]; seen as
// [batch * N rows][heads * 64 columns] a tile of one head is addressed (64 * head, batch * N + n).
inline bool make_map_rows_io(CUtensorMap* tm, int dtype, void* base, uint64_t rows, int H) {
  if (H == 0) return make_map_rows(tm, dtype, base, rows);
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)H * kD, rows / H};
  cuuint64_t strides[1] = {(cuuint64_t)H * kD * 2};
  cuuint32_t box[2] = {kD, kRows};
  cuuint32_t es[2] = {1, 1};
  return fn(tm, dtype == 1 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
            base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// 3D view (64, inner, outer) of a contiguous [outer][inner][64] array; box = (64, 1, box_outer):
// box_outer rows that are `inner` rows apart.
inline bool make_map_strided(CUtensorMap* tm, int dtype, void* base, uint64_t inner, uint64_t outer,
                             uint32_t box_outer) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {kD, inner, outer};
  cuuint64_t strides[2] = {kD * 2, inner * kD * 2};
  cuuint32_t box[3] = {kD, 1, box_outer};
  cuuint32_t es[3] = {1, 1, 1};
  return fn(tm, dtype == 1 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
            base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Strided view of an input / output tensor (rows n = inner_pos + inner * l of one head).
// H = 0: as make_map_strided, addressed (0, inner_pos, head * m + l).  H = heads: dims
// (heads * 64, inner, batch * m), addressed (64 * head, inner_pos, batch * m + l).
inline bool make_map_strided_io(CUtensorMap* tm, int dtype, void* base, uint64_t inner,
                                uint64_t outer, uint32_t box_outer, int H) {
  if (H == 0) return make_map_strided(tm, dtype, base, inner, outer, box_outer);
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)H * kD, inner, outer / H};
  cuuint64_t strides[2] = {(cuuint64_t)H * kD * 2, inner * (cuuint64_t)H * kD * 2};
  cuuint32_t box[3] = {kD, 1, box_outer};
  cuuint32_t es[3] = {1, 1, 1};
  return fn(tm, dtype == 1 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
            base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same strided view with the two outer dimensions swapped, (64, outer, inner), so that ONE box
// (64, box_outer, box_inner) brings box_inner blocks of box_outer rows each, block after block in
// shared memory: what the per-block boxes of make_map_strided_io need box_inner copies for.
// Addressed (64 * head or 0, outer index, inner index).
inline bool make_map_blocked_io(CUtensorMap* tm, int dtype, void* base, uint64_t inner,
                                uint64_t outer, uint32_t box_outer, uint32_t box_inner, int H) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t pitch = (cuuint64_t)(H ? H : 1) * kD * 2;      // bytes between consecutive rows
  cuuint64_t dims[3] = {(cuuint64_t)(H ? H : 1) * kD, H ? outer / H : outer, inner};
  cuuint64_t strides[2] = {inner * pitch, pitch};
  cuuint32_t box[3] = {kD, box_outer, box_inner};
  cuuint32_t es[3] = {1, 1, 1};
  return fn(tm, dtype == 1 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
            base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int launch(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int d, int b,
           int T, int dtype, float scale, void* ws, cudaStream_t st, int* launches);

#ifdef MA_TU_TENSOR_BASIC
template <typename T, int B>
inline int launch_t(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int T_steps,
                    int dtype, float scale, const Ws& w, cudaStream_t st, int* launches) {
  const int m = N / B;
  const uint64_t rows = (uint64_t)BH * N;
  CUtensorMap tQ, tK, tV, tAR, tAL, tYst, tALs, tYs, tQs, tARs, tOut;
  bool ok = make_map_rows(&tQ, dtype, (void*)Q, rows) && make_map_rows(&tK, dtype, (void*)K, rows) &&
            make_map_rows(&tV, dtype, (void*)V, rows) && make_map_rows(&tAR, dtype, w.aR, rows) &&
            make_map_rows(&tAL, dtype, w.aL, rows) && make_map_rows(&tYst, dtype, w.y, rows) &&
            // aL / y stores: array [BH*b (h,j)][m (k)][64]; a k-tile writes B rows j, m rows apart
            make_map_strided(&tALs, dtype, w.aL, m, (uint64_t)BH * B, B) &&
            make_map_strided(&tYs, dtype, w.y, m, (uint64_t)BH * B, B) &&
            // Q / aR / Y strided views: array [BH*m (h,l)][b (j)][64]; a j-tile touches m rows
            make_map_strided(&tQs, dtype, (void*)Q, B, (uint64_t)BH * m, B) &&
            make_map_strided(&tARs, dtype, w.aR, B, (uint64_t)BH * m, B) &&
            make_map_strided(&tOut, dtype, Y, B, (uint64_t)BH * m, B);
  if (!ok) return 7;
  if (cudaMemsetAsync(w.status, 0, kWsStatusBytes, st) != cudaSuccess) return 7;
  const int grid = BH * m / Geo<B>::kTiles;
  auto prep = [](const void* f) {
    return cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) ==
           cudaSuccess;
  };
  int n = 0;
  for (int t = 1; t <= T_steps; ++t) {
    const bool first = t == 1, last = t == T_steps;
#define MA_R(FIRST, WITHV)                                                                      \
  do {                                                                                          \
    if (!prep((const void*)r_step_tc<T, B, FIRST, WITHV>)) return 7;                            \
    r_step_tc<T, B, FIRST, WITHV><<<grid, kRows, kSmemBytes, st>>>(                             \
        FIRST ? tQ : tAR, tK, tV, tALs, tYs, w.cR, w.cL, w.status, m, scale);                   \
  } while (0)
    if (first && last) MA_R(true, true);
    else if (first) MA_R(true, false);
    else if (last) MA_R(false, true);
    else MA_R(false, false);
#undef MA_R
    ++n;
    if (last) {
      if (!prep((const void*)l_step_tc<T, B, true>)) return 7;
      l_step_tc<T, B, true><<<grid, kRows, kSmemBytes, st>>>(tQs, tAL, tYst, tOut, w.cL, w.cR,
                                                             w.status, m, scale);
    } else {
      if (!prep((const void*)l_step_tc<T, B, false>)) return 7;
      l_step_tc<T, B, false><<<grid, kRows, kSmemBytes, st>>>(tQs, tAL, tYst, tARs, w.cL, w.cR,
                                                              w.status, m, scale);
    }
    ++n;
  }
  if (cudaGetLastError() != cudaSuccess) return 7;
  *launches = n;
  return 0;
}

int launch(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int d, int b,
                  int T, int dtype, float scale, void* ws, cudaStream_t st, int* launches) {
  (void)d;
  Ws w = ws_layout(ws, BH, N);
  if (dtype == 1) {
    if (b == 128) return launch_t<__half, 128>(Q, K, V, Y, BH, N, T, dtype, scale, w, st, launches);
    return launch_t<__half, 64>(Q, K, V, Y, BH, N, T, dtype, scale, w, st, launches);
  }
  if (b == 128)
    return launch_t<__nv_bfloat16, 128>(Q, K, V, Y, BH, N, T, dtype, scale, w, st, launches);
  return launch_t<__nv_bfloat16, 64>(Q, K, V, Y, BH, N, T, dtype, scale, w, st, launches);
}

#endif  // MA_TU_TENSOR_BASIC

}  // namespace tensor
}  // namespace ma
