// Fused kernel for N = 1024 as 32 blocks of 32 (d = 64, f16/bf16): all T rounds of Eq. 7-10 and the
// Monarch multiply of Eq. 4 in ONE launch, the states alpha_L, alpha_R, y, c_L (Sec. 3
// 'Implementation') never leaving shared memory.
//
// A head of this size does not fit one SM (Q, K, V and a state are 128 KB each), so it is split by
// in-block position: within a head the whole recursion is independent across the position j (row
// (l, j) of the Monarch matrix is L[j,:,l] (x) R[:,j,:]; R[k,j,:], c_L[j,k], alpha_L[j,k,:],
// L[j,:,:], alpha_R[k,j,:], c_R[k,j], y[j,k,:] only ever read quantities with the same j, plus all
// of K and V and the 32 rows (l, j) of Q).  A CTA owns 8 positions of one head: K stays resident
// (128 KB, read once), the CTA's rows of Q and ONE state tile are 36 KB each (alpha_R and alpha_L
// replace each other in place: an R tile reads the rows (k, .) it then overwrites, an L tile the
// rows (., j)).  In the last round a block of V lands over the key block it pairs with as soon as
// that block's alpha_L is formed, and y takes eight of its rows.  No CTA exchanges anything with
// another; the four CTAs of a head read the same K and V, once from HBM and three times from L2.
//
// K, V and Q arrive by TMA (128-byte swizzle; the blocks of the Q and state tiles are 9 lines apart
// so that eight rows are conflict-free both along a block and across blocks).  Contractions are
// warp-level mma.sync m16n8k16 in f16 (bf16 inputs are converted to f16 in registers, fragment by
// fragment on their way to the tensor cores: the kernel is bound by shared-memory traffic and a
// conversion in place would add a round trip; exact for magnitudes in [6.1e-5, 65504], clamped beyond).  With 8 positions the R half-step runs transposed,
// S^T[i,j] = <K(k,i), alpha_R(k,j)> with the positions as the MMA's N: the softmax over i is a
// reduction over accumulator rows (registers, then three shuffles), the weights reach the second
// product as its B operand through movmatrix, and alpha_L^T[v,j] leaves through transposing matrix
// stores.  A warp works on two key blocks at a time.  In the L half-step two warps share a position
// (16 rows l each); for alpha_R, whose contraction runs over l, they exchange their weights through
// shared memory and each forms 16 of the 32 rows k.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "tensor_path.cuh"
#include "warp_mma.cuh"

namespace ma {
namespace jsplit {

using tensor::mbar_expect_tx;
using tensor::mbar_init;
using tensor::mbar_wait;
using tensor::tma_load_2d;
using warpmma::Mma;
using warpmma::col_sum;
using warpmma::ex2;
using warpmma::kLn2;
using warpmma::kLog2e;
using warpmma::ldsm_x4;
using warpmma::ldsm_x4_trans;
using warpmma::lg2;
using warpmma::movm_trans;
using warpmma::quad_max;
using warpmma::quad_sum;

constexpr int kN = 1024, kB = 32, kM = 32, kD = 64, kPJ = 8;   // kPJ: positions per CTA
constexpr int kThreads = 512, kWarps = 16;
constexpr int kBlkK = kB * 128;            // a key block
constexpr int kBlkQ = (kPJ + 1) * 128;     // the 8 rows (k, .) of the Q / state tile and one line of padding
constexpr int kOffK = 0;                               // [k][i][128 B]
constexpr int kOffQ = kN * 128;                        // [l][jj][128 B], blocks kBlkQ apart
constexpr int kOffS = kOffQ + kM * kBlkQ;              // state, [k][jj][128 B], blocks kBlkQ apart
constexpr int kOffP = kOffS + kM * kBlkQ;              // weights exchange: per position [32 l][32 k] f16
constexpr int kOffX = kOffP + kPJ * 2048;              // column maxima: per position [2][32] floats
constexpr int kOffC = kOffX + kPJ * 256;               // c_L, [k*8 + jj] floats
constexpr int kOffBar = kOffC + kM * kPJ * 4;          // 64 mbarriers
constexpr int kSmem = kOffBar + 64 * 8 + 1024;         // + alignment slack
static_assert(kOffQ % 1024 == 0 && kOffS % 1024 == 0 && kSmem <= 227 * 1024, "shared memory layout");

__device__ __forceinline__ float col_max(float v) {   // over the 8 row groups (lanes with equal t)
  v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 4));
  v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 8));
  return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 16));
}
__device__ __forceinline__ void stsm_x4(uint32_t saddr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1,%2,%3,%4};" ::"r"(saddr), "r"(r0),
               "r"(r1), "r"(r2), "r"(r3)
               : "memory");
}
__device__ __forceinline__ void stsm_x4_trans(uint32_t saddr, uint32_t r0, uint32_t r1, uint32_t r2,
                                              uint32_t r3) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1,%2,%3,%4};" ::"r"(saddr),
               "r"(r0), "r"(r1), "r"(r2), "r"(r3)
               : "memory");
}
// Row offsets (bytes from the 1024-byte aligned base) and the 128-byte swizzle TMA applies: the
// 16-byte chunk index is XORed with bits 7..9 of the row's address.
__device__ __forceinline__ uint32_t rk(int k, int i) { return kOffK + k * kBlkK + i * 128; }
__device__ __forceinline__ uint32_t rq(int l, int jj) { return kOffQ + l * kBlkQ + jj * 128; }
__device__ __forceinline__ uint32_t rs(int k, int jj) { return kOffS + k * kBlkQ + jj * 128; }
// y(k, j) lies in key block k at row (j + k) mod 8: conflict-free along j and along k
__device__ __forceinline__ uint32_t ry(int k, int jj) { return kOffK + k * kBlkK + ((jj + k) & 7) * 128; }
__device__ __forceinline__ uint32_t swz(uint32_t row, int c) { return row + ((c ^ ((row >> 7) & 7)) << 4); }
// exchanged weights of position jj: row l (64 bytes), 16-byte chunk c
__device__ __forceinline__ uint32_t pt(int jj, int l, int c) {
  return kOffP + jj * 2048 + l * 64 + ((c ^ ((l >> 1) & 3)) << 4);
}

template <typename TIn>
__global__ void __launch_bounds__(kThreads, 1)
monarch_jsplit32(const __grid_constant__ CUtensorMap tmQ,    // Q as [BH*N rows][64], box of 8 rows
                 const __grid_constant__ CUtensorMap tmK,    // K, box of 32 rows
                 const __grid_constant__ CUtensorMap tmV,    // V, box of 32 rows
                 TIn* __restrict__ Y, int T_steps, float scale, int* status, int H) {
  typedef __half T;
  extern __shared__ uint8_t smem_raw[];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t s0 = (uint32_t)__cvta_generic_to_shared(smem);
  float* sCL = reinterpret_cast<float*>(smem + kOffC);
  uint64_t* kbar = reinterpret_cast<uint64_t*>(smem + kOffBar);   // block k: K(k, .) and Q(k, .) have landed
  uint64_t* vbar = kbar + kM;                                     // block k: V(k, .) has landed
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int c4 = blockIdx.x;                    // which 8 of the 32 positions
  // H = 0: tensors [batch][heads][N][64], the maps see [BH * N rows][64 columns]; H = heads: tensors
  // [batch][N][heads][64], the maps see [batch * N rows][heads * 64 columns] and a head is a column
  // offset
  const int hb = H ? (int)blockIdx.y / H : (int)blockIdx.y;   // which sequence of rows
  const int x0 = H ? ((int)blockIdx.y - hb * H) * kD : 0;     // first column of the head
  const int row0 = hb * kN;                                   // the head's first row
  const float fl = scale * kLog2e;
  const int kk[2] = {warp, warp + kWarps};      // the key blocks this warp owns in the R half-steps
#ifdef MA_JSPLIT_TRACE
  long long stamps[12];
  int n_st = 0;
#define MA_STAMP() do { if (n_st < 12) stamps[n_st++] = clock64(); } while (0)
#else
#define MA_STAMP() do { } while (0)
#endif
  MA_STAMP();

  if (tid == 0) {
    for (int i = 0; i < 2 * kM; ++i) mbar_init(&kbar[i], 1);
    tensor::fence_barrier_init();
  }
  __syncthreads();
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (lane == 0) {
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      mbar_expect_tx(&kbar[kk[u]], kBlkK + kPJ * 128);
      tma_load_2d(smem + rk(kk[u], 0), &tmK, &kbar[kk[u]], x0, row0 + kk[u] * kB);
      tma_load_2d(smem + rq(kk[u], 0), &tmQ, &kbar[kk[u]], x0, row0 + kk[u] * kB + c4 * kPJ);
    }
  }
  // bf16 -> f16 of a fragment in registers (a no-op for f16 inputs)
  auto convert_frag = [&](uint32_t* a) {
    if (!Mma<TIn>::is_f16) {
      uint4 v = warpmma::to_f16x8(make_uint4(a[0], a[1], a[2], a[3]), (const TIn*)nullptr);
      a[0] = v.x; a[1] = v.y; a[2] = v.z; a[3] = v.w;
    }
  };

  uint32_t pb[2][2][2];      // the R weights of the warp's two blocks as B fragments (P^T), kept for y
  float inv_r[2][2];         // 1 / their column sums

  for (int step = 1; step <= T_steps; ++step) {
    const bool first = step == 1, last = step == T_steps;
    // ================================================================ R half-step (Eq. 7, 9, 10)
    // block k: S^T[i,j] = <K(k,i), alpha_R(k,j)> (alpha_R arrives divided by c_R), softmax over i,
    // alpha_L(k,j) = sum_i R[j,i] K(k,i), c_L(k,j) = sum_i R log R, (last) y(k,j) = sum_i R[j,i] V(k,i)
    // `which`: 0 / 1 = the warp's first / second block alone, 2 = both at a time (two independent
    // instruction streams per warp)
    auto r_pass = [&](auto which) {
      constexpr int U0 = decltype(which)::value == 1 ? 1 : 0;
      constexpr int U1 = decltype(which)::value == 0 ? 1 : 2;
      if (first) {
#pragma unroll
        for (int u = U0; u < U1; ++u) {
          if (!mbar_wait(&kbar[kk[u]], 0)) tensor::report_timeout(status, 1);
        }
        __syncwarp();
      }
      {
        // B operand: rows (k, jj) of alpha_R (L^(0) = identity: the Q rows (k, .) in the first round)
        uint32_t bq[2][2][4];
#pragma unroll
        for (int u = U0; u < U1; ++u)
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            ldsm_x4(bq[u][half], s0 + swz(first ? rq(kk[u], lane & 7) : rs(kk[u], lane & 7), (lane >> 3) + 4 * half));
            if (first) convert_frag(bq[u][half]);
          }
        float s[2][2][4];
#pragma unroll
        for (int u = U0; u < U1; ++u)
#pragma unroll
          for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int e = 0; e < 4; ++e) s[u][mt][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
#pragma unroll
          for (int u = U0; u < U1; ++u)
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
              uint32_t a[4];
              ldsm_x4(a, s0 + swz(rk(kk[u], 16 * mt + (lane & 7) + 8 * ((lane >> 3) & 1)), 2 * ks + (lane >> 4)));
              convert_frag(a);
              Mma<T>::run(s[u][mt], a, &bq[u][ks >> 1][2 * (ks & 1)]);
            }
        // column j = 2 t + e holds rows i = 16 mt + g (+ 8): softmax over i
#pragma unroll
        for (int u = U0; u < U1; ++u)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            float mx = fmaxf(fmaxf(s[u][0][e], s[u][0][e + 2]), fmaxf(s[u][1][e], s[u][1][e + 2])) * fl;
            mx = col_max(mx);
            float sum = 0.f, sz = 0.f;
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
              for (int hh = 0; hh < 2; ++hh) {
                const float z = s[u][mt][e + 2 * hh] * fl;
                const float p = ex2(z - mx);
                s[u][mt][e + 2 * hh] = p;
                sum += p;
                sz = fmaf(p, z, sz);
              }
            sum = col_sum(sum);
            sz = col_sum(sz);
            inv_r[u][e] = 1.f / sum;
            // c_L = sum R log R (natural log): ln2 * (sum p z / sum - max - log2 sum)
            if (g == 0) sCL[kk[u] * kPJ + 2 * t + e] = kLn2 * (sz * inv_r[u][e] - mx - lg2(sum));
          }
        // the weights as the second product's B operand: P^T[i, j], contraction over i
#pragma unroll
        for (int u = U0; u < U1; ++u)
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            pb[u][mt][0] = movm_trans(Mma<T>::pack(s[u][mt][0], s[u][mt][1]));
            pb[u][mt][1] = movm_trans(Mma<T>::pack(s[u][mt][2], s[u][mt][3]));
          }
        __syncwarp();
        // alpha_L^T[v, j] = sum_i K(k,i)[v] P^T[i, j]: A = the key block read transposed; the rows
        // (k, j) of alpha_L go over the alpha_R rows they were formed from (transposing stores: memory
        // row j receives column j of the accumulator tile)
#pragma unroll
        for (int vp = 0; vp < 2; ++vp) {
          float o[2][2][4];
#pragma unroll
          for (int u = U0; u < U1; ++u)
#pragma unroll
            for (int v2 = 0; v2 < 2; ++v2) {
#pragma unroll
              for (int e = 0; e < 4; ++e) o[u][v2][e] = 0.f;
#pragma unroll
              for (int is = 0; is < 2; ++is) {
                uint32_t a[4];
                ldsm_x4_trans(a, s0 + swz(rk(kk[u], 16 * is + (lane & 7) + 8 * (lane >> 4)),
                                          2 * (2 * vp + v2) + ((lane >> 3) & 1)));
                convert_frag(a);
                Mma<T>::run(o[u][v2], a, pb[u][is]);
              }
            }
#pragma unroll
          for (int u = U0; u < U1; ++u)
            stsm_x4_trans(s0 + swz(rs(kk[u], lane & 7), 4 * vp + (lane >> 3)),
                          Mma<T>::pack(o[u][0][0] * inv_r[u][0], o[u][0][1] * inv_r[u][1]),
                          Mma<T>::pack(o[u][0][2] * inv_r[u][0], o[u][0][3] * inv_r[u][1]),
                          Mma<T>::pack(o[u][1][0] * inv_r[u][0], o[u][1][1] * inv_r[u][1]),
                          Mma<T>::pack(o[u][1][2] * inv_r[u][0], o[u][1][3] * inv_r[u][1]));
        }
        if (last) {
          // the key blocks are dead: V(k, .) lands over them while the final scores are formed
          tensor::fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
#pragma unroll
            for (int u = U0; u < U1; ++u) {
              mbar_expect_tx(&vbar[kk[u]], kBlkK);
              tma_load_2d(smem + rk(kk[u], 0), &tmV, &vbar[kk[u]], x0, row0 + kk[u] * kB);
            }
          }
        }
      }
    };
    if (first) {
      // blocks are taken as they land: the first sixteen while the second sixteen are on their way
      r_pass(std::integral_constant<int, 0>());
      r_pass(std::integral_constant<int, 1>());
    } else {
      r_pass(std::integral_constant<int, 2>());
    }
    MA_STAMP();
    __syncthreads();
    MA_STAMP();

    // ================================================================ L half-step (Eq. 8, 9 / Eq. 4)
    // position jj, rows l = 16 lt ..: Z_L[l,k] = fl * <Q(l,j), alpha_L(k,j)> - c_L(k,j), softmax over k
    {
      const int jj = warp >> 1, lt = warp & 1;
      float c[4][2];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) c[nt][e] = sCL[(8 * nt + 2 * t + e) * kPJ + jj] * kLog2e;
      float s[4][4];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) s[nt][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        uint32_t a[4];
        ldsm_x4(a, s0 + swz(rq(16 * lt + (lane & 7) + 8 * ((lane >> 3) & 1), jj), 2 * ks + (lane >> 4)));
        convert_frag(a);
#pragma unroll
        for (int np = 0; np < 2; ++np) {
          uint32_t bf[4];
          ldsm_x4(bf, s0 + swz(rs(16 * np + (lane & 7) + 8 * (lane >> 4), jj), 2 * ks + ((lane >> 3) & 1)));
          Mma<T>::run(s[2 * np], a, bf);
          Mma<T>::run(s[2 * np + 1], a, bf + 2);
        }
      }
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const float z = fmaf(s[nt][2 * hh + e], fl, -c[nt][e]);
            s[nt][2 * hh + e] = z;
            mx = fmaxf(mx, z);
          }
        mx = quad_max(mx);
        float sum = 0.f;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const float p = ex2(s[nt][2 * hh + e] - mx);
            s[nt][2 * hh + e] = p;
            sum += p;
          }
        const float inv = 1.f / quad_sum(sum);
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
          for (int e = 0; e < 2; ++e) s[nt][2 * hh + e] *= inv;
      }
      if (last) {
        // Y(l,j) = sum_k L[j,k,l] y(k,j): A = the weights, rows l
        uint32_t pa[2][4];
#pragma unroll
        for (int k2 = 0; k2 < 2; ++k2) {
          pa[k2][0] = Mma<T>::pack(s[2 * k2][0], s[2 * k2][1]);
          pa[k2][1] = Mma<T>::pack(s[2 * k2][2], s[2 * k2][3]);
          pa[k2][2] = Mma<T>::pack(s[2 * k2 + 1][0], s[2 * k2 + 1][1]);
          pa[k2][3] = Mma<T>::pack(s[2 * k2 + 1][2], s[2 * k2 + 1][3]);
        }
        // y^T[v, j] = sum_i V(k,i)[v] P^T[i, j] for the warp's two blocks, V read where K was
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          if (!mbar_wait(&vbar[kk[u]], 0)) tensor::report_timeout(status, 2);
        }
        float yv[2][4][4];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
          for (int vt = 0; vt < 4; ++vt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) yv[u][vt][e] = 0.f;
#pragma unroll
            for (int is = 0; is < 2; ++is) {
              uint32_t a[4];
              ldsm_x4_trans(a, s0 + swz(rk(kk[u], 16 * is + (lane & 7) + 8 * (lane >> 4)), 2 * vt + ((lane >> 3) & 1)));
              convert_frag(a);     // V is used once: converted on its way to the tensor cores
              Mma<T>::run(yv[u][vt], a, pb[u][is]);
            }
          }
        __syncwarp();      // every row of V(k, .) is read: y(k, .) takes eight of them
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
          for (int vp = 0; vp < 2; ++vp)
            stsm_x4_trans(s0 + swz(ry(kk[u], lane & 7), 4 * vp + (lane >> 3)),
                          Mma<T>::pack(yv[u][2 * vp][0] * inv_r[u][0], yv[u][2 * vp][1] * inv_r[u][1]),
                          Mma<T>::pack(yv[u][2 * vp][2] * inv_r[u][0], yv[u][2 * vp][3] * inv_r[u][1]),
                          Mma<T>::pack(yv[u][2 * vp + 1][0] * inv_r[u][0], yv[u][2 * vp + 1][1] * inv_r[u][1]),
                          Mma<T>::pack(yv[u][2 * vp + 1][2] * inv_r[u][0], yv[u][2 * vp + 1][3] * inv_r[u][1]));
        MA_STAMP();
        __syncthreads();
        MA_STAMP();
#pragma unroll
        for (int vp = 0; vp < 4; ++vp) {          // two 8-column tiles of v per load
          float o[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
          for (int k2 = 0; k2 < 2; ++k2) {
            uint32_t bf[4];      // B[k][v] = y(k,j)[v], read transposed
            ldsm_x4_trans(bf, s0 + swz(ry(16 * k2 + (lane & 15), jj), 2 * vp + (lane >> 4)));
            Mma<T>::run(o[0], pa[k2], bf);
            Mma<T>::run(o[1], pa[k2], bf + 2);
          }
          // staged over the rows (l, j) of Q the scores were formed from (only this warp reads them)
          stsm_x4(s0 + swz(rq(16 * lt + (lane & 7) + 8 * ((lane >> 3) & 1), jj), 2 * vp + (lane >> 4)),
                  Mma<T>::pack(o[0][0], o[0][1]), Mma<T>::pack(o[0][2], o[0][3]),
                  Mma<T>::pack(o[1][0], o[1][1]), Mma<T>::pack(o[1][2], o[1][3]));
        }
        __syncwarp();
        // the warp's 16 rows (l, j) of Y are complete: 16 bytes per lane and store
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int l = 16 * lt + (lane >> 3) + 4 * r;
          const uint4 v = *reinterpret_cast<const uint4*>(smem + swz(rq(l, jj), lane & 7));
          TIn* gp = Y + ((size_t)row0 + l * kB + c4 * kPJ + jj) * (size_t)(H ? H * kD : kD) + x0 + (lane & 7) * 8;
          *reinterpret_cast<uint4*>(gp) = warpmma::from_f16x8(v, gp);
        }
      } else {
        // alpha_R(k,j) = sum_l L[j,k,l] Q(l,j) / c_R, c_R(k,j) = sum_l L[j,k,l]: the contraction
        // runs over the ROW index of the weights, which two warps share.  The result does not change
        // when column k is multiplied by any g_k > 0: g_k = 2^-(exponent of the column's largest
        // weight) keeps every column's significant weights in the normal f16 range however small
        // c_R is.  So the warps exchange their column maxima, then their scaled weights, and each
        // forms the rows k = 16 lt .. of alpha_R; c_R comes out of the same MMAs (a B operand of
        // ones), i.e. summed over the weights AS ROUNDED like the numerator.
        float* xm = reinterpret_cast<float*>(smem + kOffX + jj * 256);
        float cm[4][2];
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            cm[nt][e] = col_max(fmaxf(s[nt][e], s[nt][e + 2]));
            if (g == 0) xm[lt * 32 + 8 * nt + 2 * t + e] = cm[nt][e];
          }
        asm volatile("bar.sync %0, 64;" ::"r"(1 + jj) : "memory");
        uint32_t w[2][4];
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          float gk[2];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const float m2 = fmaxf(cm[nt][e], xm[(lt ^ 1) * 32 + 8 * nt + 2 * t + e]);
            gk[e] = m2 > 0.f ? __uint_as_float((253u << 23) - (__float_as_uint(m2) & 0x7f800000u)) : 0.f;
          }
          w[0][nt] = Mma<T>::pack(s[nt][0] * gk[0], s[nt][1] * gk[1]);
          w[1][nt] = Mma<T>::pack(s[nt][2] * gk[0], s[nt][3] * gk[1]);
        }
#pragma unroll
        for (int hh = 0; hh < 2; ++hh)
          stsm_x4(s0 + pt(jj, 16 * lt + 8 * hh + (lane & 7), lane >> 3), w[hh][0], w[hh][1], w[hh][2], w[hh][3]);
        asm volatile("bar.sync %0, 64;" ::"r"(1 + jj) : "memory");
        const int kt = lt;
        uint32_t pa[2][4];       // A[k][l] = weights transposed
#pragma unroll
        for (int ls = 0; ls < 2; ++ls)
          ldsm_x4_trans(pa[ls], s0 + pt(jj, 16 * ls + (lane & 7) + 8 * (lane >> 4), 2 * kt + ((lane >> 3) & 1)));
        float cr[4] = {0.f, 0.f, 0.f, 0.f};
        {
          const uint32_t ones[2] = {0x3C003C00u, 0x3C003C00u};
          Mma<T>::run(cr, pa[0], ones);
          Mma<T>::run(cr, pa[1], ones);
        }
        const float ic0 = cr[0] > 1e-30f ? 1.f / cr[0] : 0.f;     // row k = 16 kt + g
        const float ic1 = cr[2] > 1e-30f ? 1.f / cr[2] : 0.f;     // row k = 16 kt + g + 8
#pragma unroll
        for (int vp = 0; vp < 4; ++vp) {
          float o[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
          for (int ls = 0; ls < 2; ++ls) {
            uint32_t bf[4];   // B[l][v] = Q(l,j)[v], read transposed; two 8-column tiles
            ldsm_x4_trans(bf, s0 + swz(rq(16 * ls + (lane & 15), jj), 2 * vp + (lane >> 4)));
            convert_frag(bf);
            Mma<T>::run(o[0], pa[ls], bf);
            Mma<T>::run(o[1], pa[ls], bf + 2);
          }
          // alpha_R rows (k, j) over the alpha_L rows (both warps have formed their scores)
          stsm_x4(s0 + swz(rs(16 * kt + (lane & 7) + 8 * ((lane >> 3) & 1), jj), 2 * vp + (lane >> 4)),
                  Mma<T>::pack(o[0][0] * ic0, o[0][1] * ic0), Mma<T>::pack(o[0][2] * ic1, o[0][3] * ic1),
                  Mma<T>::pack(o[1][0] * ic0, o[1][1] * ic0), Mma<T>::pack(o[1][2] * ic1, o[1][3] * ic1));
        }
      }
    }
    MA_STAMP();
    __syncthreads();
    MA_STAMP();
  }
#ifdef MA_JSPLIT_TRACE
  if (blockIdx.x == 0 && blockIdx.y == 0 && lane == 0) {
    long long* out = reinterpret_cast<long long*>(Y) + 16384 + warp * 16;   // probe builds only
    for (int i = 0; i < n_st; ++i) out[i] = stamps[i] - stamps[0];
  }
#endif
#undef MA_STAMP
}

inline bool supported(int N, int d, int b, int m, int dtype, int BH) {
  return (dtype == 1 || dtype == 2) && N == kN && d == kD && b == kB && m == kM && BH <= 65535;
}

// `status`: device word that a bounded wait which ran out sets (never cleared by the kernel).
int launch(const void* Q, const void* K, const void* V, void* Y, int BH, int T, int dtype, float scale,
           int* status, cudaStream_t st, int H = 0);

#ifdef MA_TU_FUSED_JSPLIT
struct Maps {
  const void *q = nullptr, *k = nullptr, *v = nullptr;
  int BH = 0, dtype = 0, dev = -1, H = 0;
  CUtensorMap tmQ, tmK, tmV;
};
inline bool make_map(CUtensorMap* tm, int dtype, const void* base, uint64_t rows, uint32_t box_rows, int H) {
  tensor::EncodeTiledFn fn = tensor::encode_fn();
  if (!fn) return false;
  const uint64_t cols = H ? (uint64_t)H * kD : kD;
  if (H) rows /= H;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {kD, box_rows};
  cuuint32_t es[2] = {1, 1};
  return fn(tm, dtype == 1 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
            const_cast<void*>(base), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename TIn>
inline int launch_t(const Maps& mp, void* Y, int BH, int T, float scale, int* status, cudaStream_t st,
                    int dev, int H) {
  auto kern = monarch_jsplit32<TIn>;
  static bool prepared[64] = {};
  if (!prepared[dev]) {
    if (cudaFuncSetAttribute((const void*)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) != cudaSuccess)
      return 7;
    prepared[dev] = true;
  }
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kB / kPJ, BH);     // the four CTAs of a head are neighbours: they share K and V in L2
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmem;
  cfg.stream = st;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, mp.tmQ, mp.tmK, mp.tmV, (TIn*)Y, T, scale, status, H) == cudaSuccess ? 0 : 7;
}

int launch(const void* Q, const void* K, const void* V, void* Y, int BH, int T, int dtype, float scale,
           int* status, cudaStream_t st, int H) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 7;
  // the tensor maps of the last few (Q, K, V) triples are kept: encoding three maps costs more host
  // time than the launch itself
  static thread_local Maps cache[4];
  static thread_local int next = 0;
  const Maps* mp = nullptr;
  for (int i = 0; i < 4; ++i)
    if (cache[i].q == Q && cache[i].k == K && cache[i].v == V && cache[i].BH == BH && cache[i].dtype == dtype &&
        cache[i].dev == dev && cache[i].H == H)
      mp = &cache[i];
  if (!mp) {
    Maps& m = cache[next];
    next = (next + 1) % 4;
    m.dev = -1;
    const uint64_t rows = (uint64_t)BH * kN;
    if (!make_map(&m.tmQ, dtype, Q, rows, kPJ, H) || !make_map(&m.tmK, dtype, K, rows, kB, H) ||
        !make_map(&m.tmV, dtype, V, rows, kB, H))
      return 7;
    m.q = Q; m.k = K; m.v = V; m.BH = BH; m.dtype = dtype; m.dev = dev; m.H = H;
    mp = &m;
  }
  if (dtype == 1) return launch_t<__half>(*mp, Y, BH, T, scale, status, st, dev, H);
  return launch_t<__nv_bfloat16>(*mp, Y, BH, T, scale, status, st, dev, H);
}
#endif  // MA_TU_FUSED_JSPLIT

}  // namespace jsplit
}  // namespace ma
