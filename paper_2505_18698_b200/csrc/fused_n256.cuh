// Fully fused per-head kernel for short sequences: N = 256, m = b = 16, d = 64, f16/bf16.
//
// One CTA (8 warps) per (batch, head).  Q, K, V are read from HBM once into shared memory, every
// half-step of all T rounds runs out of shared memory and registers, and Y is written once: HBM
// traffic is exactly one read of Q, K, V and one write of Y (Sec. 3: Theta(N d) IO).  The block
// factors R (16x16 per key block) and L (16x16 per in-block position) live only in registers;
// the states alpha_L, alpha_R, y (Sec. 3 'Implementation') stay in shared memory.
//
// Arithmetic is f16 x f16 -> fp32 whatever the input type: bf16 inputs are converted to f16 when
// they are copied into shared memory (exact for magnitudes in [6.1e-5, 65504]; larger ones are
// clamped) and the result is converted back on the way out.  The dominant error of a 16-bit
// pipeline is the rounding of the alpha_L state (it feeds logits of size ~100), and f16 carries
// three more mantissa bits than bf16 there.
//
// The 16x16x64 contractions are warp-level mma.sync m16n8k16 (a 16-row block does not fill a
// tcgen05 tile).  Warp w owns key blocks k = 2w, 2w+1 in an R half-step and in-block positions
// j = 2w, 2w+1 in an L half-step; the permutation between the two is the index arithmetic of the
// shared-memory rows ([k][j] vs [j][k]).  On the last round alpha_L and y overwrite K and V (dead
// by then) and Y overwrites the rows of Q a warp has finished with, so T = 1 needs 98 KB and two
// CTAs share an SM (one loads while the other computes).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ma {
namespace fused {

constexpr int kN = 256, kB = 16, kD = 64, kThreads = 256;
constexpr int kTile = kN * kD * 2;                       // 32 KB
constexpr int kSmemT1 = 3 * kTile + 2048 + 1024;         // Q, K, V, cL, cR (+ alignment slack)
constexpr int kSmemTn = 5 * kTile + 2048 + 1024;         // + alpha_L, alpha_R of the earlier rounds
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Shared-memory address of element (row, col) of a [256][64] 16-bit tile.  16-byte chunks are
// XOR-swizzled with the row's position inside its 16-row block AND with the block index, so that
// fragment loads are conflict-free both over 8 consecutive rows and over 8 rows 16 apart.
__device__ __forceinline__ uint32_t swz(int row, int col) {
  const int chunk = (col >> 3) ^ (row & 7) ^ ((row >> 4) & 7);
  return (uint32_t)(row * 128 + (chunk << 4) + ((col & 7) << 1));
}

template <typename T> struct Mma;
template <> struct Mma<__half> {
  static __device__ __forceinline__ void run(float* c, const uint32_t* a, const uint32_t* b) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
  }
  static constexpr bool is_f16 = true;
  static __device__ __forceinline__ uint32_t pack(float x, float y) {
    __half2 h = __floats2half2_rn(x, y);
    return *reinterpret_cast<uint32_t*>(&h);
  }
  static __device__ __forceinline__ float2 unpack(uint32_t u) {
    return __half22float2(*reinterpret_cast<__half2*>(&u));
  }
};
template <> struct Mma<__nv_bfloat16> {
  static __device__ __forceinline__ void run(float* c, const uint32_t* a, const uint32_t* b) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
  }
  static constexpr bool is_f16 = false;
  static __device__ __forceinline__ uint32_t pack(float x, float y) {
    __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
    return *reinterpret_cast<uint32_t*>(&h);
  }
  static __device__ __forceinline__ float2 unpack(uint32_t u) {
    return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
  }
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t lds32(const uint8_t* base, uint32_t off) {
  return *reinterpret_cast<const uint32_t*>(base + off);
}
// B fragment (k = 16 rows, n = 8 columns) of a matrix stored [k rows][n contiguous]: transposing
// 8x8 loads.  `row_of(kk)` gives the tile row of contraction index kk, col0 the first n.
__device__ __forceinline__ void ldsm_x2_trans(uint32_t* b, uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];"
               : "=r"(b[0]), "=r"(b[1])
               : "r"(saddr));
}
__device__ __forceinline__ void ldsm_x4(uint32_t* r, uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(saddr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t* r, uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(saddr));
}
__device__ __forceinline__ uint32_t movm_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
__device__ __forceinline__ float quad_max(float v) {
  v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
  return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
}
__device__ __forceinline__ float quad_sum(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  return v + __shfl_xor_sync(0xffffffffu, v, 2);
}
__device__ __forceinline__ float col_sum(float v) {   // over the 8 row groups (lanes with equal t)
  v += __shfl_xor_sync(0xffffffffu, v, 4);
  v += __shfl_xor_sync(0xffffffffu, v, 8);
  return v + __shfl_xor_sync(0xffffffffu, v, 16);
}

__device__ __forceinline__ uint4 to_f16x8(uint4 v, const __half*) { return v; }
__device__ __forceinline__ uint4 to_f16x8(uint4 v, const __nv_bfloat16*) {
  uint32_t* w = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float lo = fminf(fmaxf(__uint_as_float(w[i] << 16), -65504.f), 65504.f);
    const float hi = fminf(fmaxf(__uint_as_float(w[i] & 0xffff0000u), -65504.f), 65504.f);
    w[i] = Mma<__half>::pack(lo, hi);
  }
  return v;
}
__device__ __forceinline__ uint4 from_f16x8(uint4 v, __half*) { return v; }
__device__ __forceinline__ uint4 from_f16x8(uint4 v, __nv_bfloat16*) {
  uint32_t* w = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = Mma<__half>::unpack(w[i]);
    w[i] = Mma<__nv_bfloat16>::pack(f.x, f.y);
  }
  return v;
}

template <typename TIn>
__global__ void __launch_bounds__(kThreads, 2)
monarch_fused_n256(const TIn* __restrict__ Q, const TIn* __restrict__ K, const TIn* __restrict__ V,
                   TIn* __restrict__ Y, int T_steps, float scale) {
  typedef __half T;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;
  uint8_t* sK = smem + kTile;
  uint8_t* sV = smem + 2 * kTile;
  float* sCL = reinterpret_cast<float*>(smem + 3 * kTile);          // [j][k]
  float* sCR = sCL + 256;                                            // [k][j]
  uint8_t* sALx = smem + 3 * kTile + 2048;                           // T > 1 only
  uint8_t* sAR = sALx + kTile;                                       // T > 1 only
  const uint32_t sQ_u = (uint32_t)__cvta_generic_to_shared(sQ);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const size_t head = (size_t)blockIdx.x * kN * kD;

  // ---- load Q, K, V: 16-byte asynchronous copies into the swizzled layout
  {
    const TIn* src[3] = {Q + head, K + head, V + head};
#pragma unroll
    for (int a = 0; a < 3; ++a) {
      const uint32_t dst0 = sQ_u + a * kTile;
      for (int idx = tid; idx < kN * 8; idx += kThreads) {
        const int row = idx >> 3, ch = idx & 7;
        const TIn* gp = src[a] + (size_t)row * kD + ch * 8;
        if (sizeof(TIn) == 2 && Mma<TIn>::is_f16) {
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst0 + swz(row, ch * 8)),
                       "l"(gp));
        } else {
          const uint4 v = __ldg(reinterpret_cast<const uint4*>(gp));
          *reinterpret_cast<uint4*>(smem + a * kTile + swz(row, ch * 8)) = to_f16x8(v, gp);
        }
      }
    }
    asm volatile("cp.async.commit_group;");
    asm volatile("cp.async.wait_group 0;");
    __syncthreads();
  }

  const float fl = scale * kLog2e;
  for (int step = 1; step <= T_steps; ++step) {
    const bool first = step == 1, last = step == T_steps;
    // ================================================================ R half-step (Eq. 7, 9, 10)
    const uint8_t* sA = first ? sQ : sAR;          // alpha_R[k][j][:] (= Q rows when L = identity)
    const uint32_t sA_u = (uint32_t)__cvta_generic_to_shared(sA);
    const uint32_t sK_u = sQ_u + kTile, sV_u = sQ_u + 2 * kTile;
    uint32_t outL[2][8][2], outY[2][8][2];          // packed alpha_L / y rows g and g+8, per v block
#pragma unroll
    for (int kt = 0; kt < 2; ++kt) {
      const int k = 2 * warp + kt, r0 = 16 * k;
      float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        // A: 16 rows x 16 k as four 8x8 matrices (rows 0-7 / 8-15, k 0-7 / 8-15), one ldmatrix;
        // B: both 8-column tiles of K (stored [i][v]) likewise.
        uint32_t a[4], b[4];
        ldsm_x4(a, sA_u + swz(r0 + (lane & 7) + ((lane >> 3) & 1) * 8, 16 * ks + (lane >> 4) * 8));
        ldsm_x4(b, sK_u + swz(r0 + (lane & 7) + (lane >> 4) * 8, 16 * ks + ((lane >> 3) & 1) * 8));
        Mma<T>::run(s[0], a, b);
        Mma<T>::run(s[1], a, b + 2);
      }
      // rows j = g (c0, c1) and j = g + 8 (c2, c3); columns i = 8 nt + 2t, +1
      float inv_s[2], pa_f[2][4];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int j = g + 8 * h;
        float f = fl;
        if (!first) {
          const float c = sCR[k * 16 + j];
          f = c > 1e-30f ? fl / c : 0.f;
        }
        const float z0 = s[0][2 * h] * f, z1 = s[0][2 * h + 1] * f;
        const float z2 = s[1][2 * h] * f, z3 = s[1][2 * h + 1] * f;
        const float mx = quad_max(fmaxf(fmaxf(z0, z1), fmaxf(z2, z3)));
        const float p0 = ex2(z0 - mx), p1 = ex2(z1 - mx), p2 = ex2(z2 - mx), p3 = ex2(z3 - mx);
        const float sum = quad_sum((p0 + p1) + (p2 + p3));
        const float sz = quad_sum(fmaf(p0, z0, p1 * z1) + fmaf(p2, z2, p3 * z3));
        inv_s[h] = 1.f / sum;
        // c_L = sum R log R (natural log): ln2 * (sum p z / sum - max - log2 sum)
        if (t == 0) sCL[j * 16 + k] = kLn2 * (sz * inv_s[h] - mx - lg2(sum));
        pa_f[h][0] = p0; pa_f[h][1] = p1; pa_f[h][2] = p2; pa_f[h][3] = p3;
      }
      uint32_t pa[4];
      pa[0] = Mma<T>::pack(pa_f[0][0], pa_f[0][1]);
      pa[1] = Mma<T>::pack(pa_f[1][0], pa_f[1][1]);
      pa[2] = Mma<T>::pack(pa_f[0][2], pa_f[0][3]);
      pa[3] = Mma<T>::pack(pa_f[1][2], pa_f[1][3]);
#pragma unroll
      for (int np = 0; np < 4; ++np) {     // two 8-column tiles of v per transposing ldmatrix
        uint32_t b[4];
        ldsm_x4_trans(b, sK_u + swz(r0 + (lane & 15), 16 * np + (lane >> 4) * 8));
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          float o[4] = {0.f, 0.f, 0.f, 0.f};
          Mma<T>::run(o, pa, b + 2 * q);
          outL[kt][2 * np + q][0] = Mma<T>::pack(o[0] * inv_s[0], o[1] * inv_s[0]);
          outL[kt][2 * np + q][1] = Mma<T>::pack(o[2] * inv_s[1], o[3] * inv_s[1]);
        }
        if (last) {
          ldsm_x4_trans(b, sV_u + swz(r0 + (lane & 15), 16 * np + (lane >> 4) * 8));
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            float y[4] = {0.f, 0.f, 0.f, 0.f};
            Mma<T>::run(y, pa, b + 2 * q);
            outY[kt][2 * np + q][0] = Mma<T>::pack(y[0] * inv_s[0], y[1] * inv_s[0]);
            outY[kt][2 * np + q][1] = Mma<T>::pack(y[2] * inv_s[1], y[3] * inv_s[1]);
          }
        }
      }
    }
    __syncthreads();   // every warp is done with K (and V): alpha_L / y may take their place
    uint8_t* sAL = last ? sK : sALx;               // alpha_L[j][k][:]; y[j][k][:] goes over V
#pragma unroll
    for (int kt = 0; kt < 2; ++kt) {
      const int k = 2 * warp + kt;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const uint32_t off = swz(16 * (g + 8 * h) + k, 8 * nt + 2 * t);
          *reinterpret_cast<uint32_t*>(sAL + off) = outL[kt][nt][h];
          if (last) *reinterpret_cast<uint32_t*>(sV + off) = outY[kt][nt][h];
        }
      }
    }
    __syncthreads();

    // ================================================================ L half-step (Eq. 8, 9 / Eq. 4)
    const uint32_t sAL_u = (uint32_t)__cvta_generic_to_shared(sAL);
#pragma unroll
    for (int jt = 0; jt < 2; ++jt) {
      const int j = 2 * warp + jt;
      float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        // A: rows l of Qb[j] are tile rows 16 l + j; B: alpha_L[j][k][:] rows 16 j + k
        uint32_t a[4], b[4];
        ldsm_x4(a, sQ_u + swz(16 * ((lane & 7) + ((lane >> 3) & 1) * 8) + j, 16 * ks + (lane >> 4) * 8));
        ldsm_x4(b, sAL_u + swz(16 * j + (lane & 7) + (lane >> 4) * 8, 16 * ks + ((lane >> 3) & 1) * 8));
        Mma<T>::run(s[0], a, b);
        Mma<T>::run(s[1], a, b + 2);
      }
      // rows l = g, g + 8; columns k = 8 nt + 2t, +1.  Z_L = scale * S' - c_L[j][k]
      const float c0 = sCL[j * 16 + 2 * t] * kLog2e, c1 = sCL[j * 16 + 2 * t + 1] * kLog2e;
      const float c2 = sCL[j * 16 + 8 + 2 * t] * kLog2e, c3 = sCL[j * 16 + 8 + 2 * t + 1] * kLog2e;
      float p[2][4], inv_s[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const float z0 = fmaf(s[0][2 * h], fl, -c0), z1 = fmaf(s[0][2 * h + 1], fl, -c1);
        const float z2 = fmaf(s[1][2 * h], fl, -c2), z3 = fmaf(s[1][2 * h + 1], fl, -c3);
        const float mx = quad_max(fmaxf(fmaxf(z0, z1), fmaxf(z2, z3)));
        p[h][0] = ex2(z0 - mx); p[h][1] = ex2(z1 - mx); p[h][2] = ex2(z2 - mx); p[h][3] = ex2(z3 - mx);
        inv_s[h] = 1.f / quad_sum((p[h][0] + p[h][1]) + (p[h][2] + p[h][3]));
      }
      if (last) {
        // Y[16 l + j][:] = sum_k L[j,k,l] y[j][k][:]   (A = P' rows l, B = y[j] read transposed)
        uint32_t pa[4];
        pa[0] = Mma<T>::pack(p[0][0], p[0][1]);
        pa[1] = Mma<T>::pack(p[1][0], p[1][1]);
        pa[2] = Mma<T>::pack(p[0][2], p[0][3]);
        pa[3] = Mma<T>::pack(p[1][2], p[1][3]);
        uint32_t out[8][2];
#pragma unroll
        for (int np = 0; np < 4; ++np) {
          uint32_t b[4];
          ldsm_x4_trans(b, sV_u + swz(16 * j + (lane & 15), 16 * np + (lane >> 4) * 8));
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            float o[4] = {0.f, 0.f, 0.f, 0.f};
            Mma<T>::run(o, pa, b + 2 * q);
            out[2 * np + q][0] = Mma<T>::pack(o[0] * inv_s[0], o[1] * inv_s[0]);
            out[2 * np + q][1] = Mma<T>::pack(o[2] * inv_s[1], o[3] * inv_s[1]);
          }
        }
        // only this warp reads the rows 16 l + j of Q, and it has: Y takes their place
        __syncwarp();
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          *reinterpret_cast<uint32_t*>(sQ + swz(16 * g + j, 8 * nt + 2 * t)) = out[nt][0];
          *reinterpret_cast<uint32_t*>(sQ + swz(16 * (g + 8) + j, 8 * nt + 2 * t)) = out[nt][1];
        }
      } else {
        // alpha_R[k][j][:] = sum_l L[j,k,l] Qb[j][l][:], c_R[k][j] = sum_l L[j,k,l]: the
        // contraction runs over the ROW index of P', so the A fragments are its transpose.
        float pn[2][4];
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int e = 0; e < 4; ++e) pn[h][e] = p[h][e] * inv_s[h];
        // alpha_R / c_R does not change when column k of the weights is multiplied by any g_k > 0.
        // g_k = 2^-(exponent of the column's largest weight) keeps every column's significant
        // weights in the normal f16 range however small c_R is (it can be 1e-8).
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float cm = fmaxf(pn[0][e], pn[1][e]);
          cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 4));
          cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 8));
          cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 16));
          // power of two not above 1/cm (exact scaling); columns that are all zero stay zero
          const float gk = cm > 0.f ? __uint_as_float((253u << 23) - (__float_as_uint(cm) & 0x7f800000u)) : 0.f;
          pn[0][e] *= gk;
          pn[1][e] *= gk;
        }
        const uint32_t t00 = Mma<T>::pack(pn[0][0], pn[0][1]), t10 = Mma<T>::pack(pn[1][0], pn[1][1]);
        const uint32_t t01 = Mma<T>::pack(pn[0][2], pn[0][3]), t11 = Mma<T>::pack(pn[1][2], pn[1][3]);
        uint32_t pa[4];
        pa[0] = movm_trans(t00);   // rows k 0-7,  cols l 0-7
        pa[1] = movm_trans(t01);   // rows k 8-15, cols l 0-7
        pa[2] = movm_trans(t10);   // rows k 0-7,  cols l 8-15
        pa[3] = movm_trans(t11);   // rows k 8-15, cols l 8-15
        // column sums of the normalised P' AS ROUNDED to 16 bit: alpha_R / c_R is a weighted mean
        // of Q rows, and it stays one only if numerator (the MMA below) and denominator see the
        // same weights -- c_R can be 1e-6, where rounding the weights changes them a lot.
        const float2 u00 = Mma<T>::unpack(t00), u10 = Mma<T>::unpack(t10);
        const float2 u01 = Mma<T>::unpack(t01), u11 = Mma<T>::unpack(t11);
        const float cs0 = col_sum(u00.x + u10.x), cs1 = col_sum(u00.y + u10.y);
        const float cs2 = col_sum(u01.x + u11.x), cs3 = col_sum(u01.y + u11.y);
        if (g == 0) {
          sCR[(2 * t) * 16 + j] = cs0;
          sCR[(2 * t + 1) * 16 + j] = cs1;
          sCR[(8 + 2 * t) * 16 + j] = cs2;
          sCR[(8 + 2 * t + 1) * 16 + j] = cs3;
        }
        __syncwarp();
        // alpha_R is stored already divided by c_R (in fp32, before rounding): c_R can be tiny for
        // peaky attention and the un-normalised state would leave the 16-bit range.
        const float cr0 = sCR[g * 16 + j], cr1 = sCR[(g + 8) * 16 + j];
        const float ic0 = cr0 > 1e-30f ? 1.f / cr0 : 0.f, ic1 = cr1 > 1e-30f ? 1.f / cr1 : 0.f;
        __syncwarp();
        if (t == 0) {          // the next R half-step divides by c_R: it is 1 from now on
          sCR[g * 16 + j] = 1.f;
          sCR[(g + 8) * 16 + j] = 1.f;
        }
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          float o[4] = {0.f, 0.f, 0.f, 0.f};
          uint32_t b[2];   // B[kk = l][n = v] = Qb[j][l][v]: tile rows 16 l + j, read transposed
          ldsm_x2_trans(b, sQ_u + swz(16 * (lane & 15) + j, 8 * nt));
          Mma<T>::run(o, pa, b);
          // rows k = g, g + 8 -> alpha_R tile rows 16 k + j
          *reinterpret_cast<uint32_t*>(sAR + swz(16 * g + j, 8 * nt + 2 * t)) =
              Mma<T>::pack(o[0] * ic0, o[1] * ic0);
          *reinterpret_cast<uint32_t*>(sAR + swz(16 * (g + 8) + j, 8 * nt + 2 * t)) =
              Mma<T>::pack(o[2] * ic1, o[3] * ic1);
        }
      }
    }
    __syncthreads();
  }

  // ---- Y sits where Q was: coalesced 16-byte copies out
  TIn* out = Y + head;
  for (int idx = tid; idx < kN * 8; idx += kThreads) {
    const int row = idx >> 3, ch = idx & 7;
    const uint4 v = *reinterpret_cast<const uint4*>(sQ + swz(row, ch * 8));
    TIn* gp = out + (size_t)row * kD + ch * 8;
    *reinterpret_cast<uint4*>(gp) = from_f16x8(v, gp);
  }
}

inline bool supported(int N, int d, int b, int m, int dtype, int BH) {
  (void)BH;
  return (dtype == 1 || dtype == 2) && N == kN && d == kD && b == kB && m == kB;
}

inline int launch(const void* Q, const void* K, const void* V, void* Y, int BH, int T, int dtype,
                  float scale, cudaStream_t st) {
  const int smem = T == 1 ? kSmemT1 : kSmemTn;
  if (dtype == 1) {
    auto kern = monarch_fused_n256<__half>;
    if (cudaFuncSetAttribute((const void*)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTn) != cudaSuccess) return 7;
    kern<<<BH, kThreads, smem, st>>>((const __half*)Q, (const __half*)K, (const __half*)V, (__half*)Y, T, scale);
  } else {
    auto kern = monarch_fused_n256<__nv_bfloat16>;
    if (cudaFuncSetAttribute((const void*)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTn) != cudaSuccess) return 7;
    kern<<<BH, kThreads, smem, st>>>((const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, (const __nv_bfloat16*)V, (__nv_bfloat16*)Y, T, scale);
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 7;
}

}  // namespace fused
}  // namespace ma
