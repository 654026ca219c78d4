// Fused fp32 kernel for short sequences: all T rounds of Eq. 7-10 and the Monarch multiply of Eq. 4
// in ONE launch, fp32 arithmetic and fp32 states in shared memory (the accuracy of the generic
// kernels without their 2T launches and their round trips through the workspace).
//
// Within a head the whole recursion is independent across the in-block position j: row (l, j) of
// the Monarch matrix is L[j,:,l] (x) R[:,j,:], and R[k,j,:], c_L[j,k], alpha_L[j,k,:], L[j,:,:],
// alpha_R[k,j,:], c_R[k,j], y[j,k,:] only ever read quantities with the SAME j, plus K, V and the m
// rows (l, j) of Q (Eq. 7-10: the softmax over i and the sum over i couple a key block, the softmax
// over k and the sum over l couple a position).  A CTA therefore owns a set J of positions of one
// head, loads all of K and V and its own rows of Q once, and runs every half-step for its J with
// no exchange with other CTAs.  A single small head (one SM's worth of work or less) is spread over
// up to b CTAs this way; with many heads a CTA takes all b positions of a head and K, V are read
// once.
//
// Inside the CTA a warp takes one (block, position) pair at a time: lanes over the b keys (R) or the
// m blocks (L) for the scores and the softmax (warp shuffles), then lanes over the d columns for the
// second product.  Rows are padded to d + 1 floats, so a lane per row reads conflict-free.
#pragma once
#include <cuda_runtime.h>

#include "generic_kernels.cuh"

namespace ma {
namespace ffused {

using generic::io_off;
using generic::ld_as_float;
using generic::st_from_float;
using generic::warp_max;
using generic::warp_sum;

constexpr int kThreads = 512, kWarps = kThreads / 32, kMaxSmem = 227 * 1024;

// Shared-memory floats: K and V (all rows), then for the CTA's JT positions the m rows of Q,
// alpha_L, alpha_R, y, the vectors c_L, c_R, the normalised L weights, and per-warp scratch.
__host__ __device__ inline size_t smem_floats(int N, int d, int b, int m, int JT) {
  const size_t dp = d + 1;
  const size_t mx = b > m ? b : m;
  return 2 * (size_t)N * dp + 4 * (size_t)JT * m * dp + 2 * (size_t)JT * m + (size_t)JT * m * (m + 1) +
         (size_t)kWarps * (mx + d);
}

// Positions per CTA: all b of a head when there are heads enough to fill the GPU, fewer (down to
// one) when there are not, as long as the CTA's tiles fit shared memory.  0: does not fit at all.
inline int positions_per_cta(int N, int d, int b, int m, int BH, int num_sms) {
  int jt = b;
  while (jt > 1 && (long long)BH * ((b + jt - 1) / jt) < 2LL * num_sms) jt = (jt + 1) / 2;
  while (jt >= 1 && smem_floats(N, d, b, m, jt) * 4 > (size_t)kMaxSmem) --jt;
  return jt;
}
inline bool supported(int N, int d, int b, int m) {
  return b <= 1024 && m <= 1024 && smem_floats(N, d, b, m, 1) * 4 <= (size_t)kMaxSmem;
}

template <typename TIn>
__global__ void __launch_bounds__(kThreads, 1)
monarch_fused_f32(const TIn* __restrict__ Q, const TIn* __restrict__ K, const TIn* __restrict__ V,
                  TIn* __restrict__ Y, int N, int d, int b, int m, int T_steps, float scale,
                  int n_valid, int H, int JT, float* __restrict__ row_lse) {
  extern __shared__ float smem[];
  generic::grid_dependency_sync();
  const int h = blockIdx.y, j0 = blockIdx.x * JT, nj = min(JT, b - j0);
  const int dp = d + 1, mp = m + 1;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  float* Ks = smem;                                   // [N][dp]
  float* Vs = Ks + (size_t)N * dp;                    // [N][dp]
  float* Qs = Vs + (size_t)N * dp;                    // [jj][l][dp]: row (l, j0 + jj) of Q
  float* aLs = Qs + (size_t)JT * m * dp;              // [jj][k][dp]
  float* aRs = aLs + (size_t)JT * m * dp;             // [jj][k][dp]
  float* ys = aRs + (size_t)JT * m * dp;              // [jj][k][dp]
  float* cLs = ys + (size_t)JT * m * dp;              // [jj][k]
  float* cRs = cLs + (size_t)JT * m;                  // [jj][k]
  float* Ls = cRs + (size_t)JT * m;                   // [jj][l][mp]: normalised L weights
  float* wbuf = Ls + (size_t)JT * m * mp;
  const int mx = b > m ? b : m;
  float* zs = wbuf + (size_t)warp * (mx + d);         // per warp: weights of the current row
  (void)zs;

  // Loads: 16 bytes per thread and several of them in flight (a CTA's share of a small problem is
  // latency-bound: K and V are 2 x N x d elements for as little as one position's work).
  constexpr int kVec = 16 / (int)sizeof(TIn);         // elements per 16-byte load
  if (d % kVec == 0) {
    const int dv = d / kVec;
    auto put = [&](float* dst, const uint4& u) {
      const TIn* e = reinterpret_cast<const TIn*>(&u);
#pragma unroll
      for (int c = 0; c < kVec; ++c) dst[c] = ld_as_float(e + c);
    };
#pragma unroll 4
    for (int e = tid; e < N * dv; e += kThreads) {
      const int n = e / dv, v = (e - n * dv) * kVec;
      const size_t off = io_off(h, n, N, d, H) + v;
      const uint4 kq = *reinterpret_cast<const uint4*>(K + off);
      const uint4 vq = *reinterpret_cast<const uint4*>(V + off);
      put(Ks + n * dp + v, kq);
      put(Vs + n * dp + v, vq);
    }
#pragma unroll 4
    for (int e = tid; e < nj * m * dv; e += kThreads) {
      const int r = e / dv, v = (e - r * dv) * kVec;  // r = jj * m + l
      const int jj = r / m, l = r - jj * m;
      const uint4 qq = *reinterpret_cast<const uint4*>(Q + io_off(h, l * b + j0 + jj, N, d, H) + v);
      put(Qs + r * dp + v, qq);
    }
  } else {
    for (int e = tid; e < N * d; e += kThreads) {
      const int n = e / d, v = e - n * d;
      const size_t off = io_off(h, n, N, d, H) + v;
      Ks[n * dp + v] = ld_as_float(K + off);
      Vs[n * dp + v] = ld_as_float(V + off);
    }
    for (int e = tid; e < nj * m * d; e += kThreads) {
      const int r = e / d, v = e - r * d;             // r = jj * m + l
      const int jj = r / m, l = r - jj * m;
      Qs[r * dp + v] = ld_as_float(Q + io_off(h, l * b + j0 + jj, N, d, H) + v);
    }
  }
  __syncthreads();

  for (int step = 1; step <= T_steps; ++step) {
    const bool first = step == 1, last = step == T_steps;
    // ---------------------------------------------------------------- R half-step (Eq. 7, 9, 10)
    // pair (k, jj): Z_R[i] = scale * <alpha_R(k,j), K(k,i)> / c_R(k,j); R = softmax_i Z_R;
    // alpha_L(j,k) = sum_i R[i] K(k,i); c_L(j,k) = sum_i R log R; (last) y(j,k) = sum_i R[i] V(k,i)
    for (int p = warp; p < m * nj; p += kWarps) {
      const int k = p / nj, jj = p - k * nj, r = jj * m + k;
      // L^(0) = identity: alpha_R = the Q row (k, j), c_R = 1
      const float* a = first ? Qs + (size_t)r * dp : aRs + (size_t)r * dp;
      float inv_c = 1.f;
      if (!first) {
        const float c = cRs[r];
        inv_c = c > 1e-30f ? 1.f / c : 0.f;            // c_R underflow: uniform row (Z_R = 0)
      }
      const float f = scale * inv_c;
      float zmax = -INFINITY;
      for (int i = lane; i < b; i += 32) {
        const float* kr = Ks + (size_t)(k * b + i) * dp;
        float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
        int v = 0;
        for (; v + 3 < d; v += 4) {
          acc0 = fmaf(a[v], kr[v], acc0);
          acc1 = fmaf(a[v + 1], kr[v + 1], acc1);
          acc2 = fmaf(a[v + 2], kr[v + 2], acc2);
          acc3 = fmaf(a[v + 3], kr[v + 3], acc3);
        }
        for (; v < d; ++v) acc0 = fmaf(a[v], kr[v], acc0);
        // padding mask (App. C.3, post-padding): key columns b k + i >= n_valid get -inf
        const float z = (k * b + i < n_valid) ? ((acc0 + acc1) + (acc2 + acc3)) * f : -INFINITY;
        zs[i] = z;
        zmax = fmaxf(zmax, z);
      }
      zmax = warp_max(zmax);
      float s = 0.f, sz = 0.f;
      for (int i = lane; i < b; i += 32) {
        const float z = zs[i];
        const bool valid = z > -INFINITY;
        const float pw = valid ? expf(z - zmax) : 0.f;
        zs[i] = pw;
        s += pw;
        if (valid) sz = fmaf(pw, z, sz);               // 0 log 0 = 0 for masked keys
      }
      s = warp_sum(s);
      sz = warp_sum(sz);
      __syncwarp();
      const float inv_s = 1.f / s;
      for (int v = lane; v < d; v += 32) {
        float acc = 0.f, accv = 0.f;
        const float* kc = Ks + (size_t)k * b * dp + v;
        const float* vc = Vs + (size_t)k * b * dp + v;
        for (int i = 0; i < b; ++i) {
          const float pw = zs[i];
          acc = fmaf(pw, kc[(size_t)i * dp], acc);
          if (last) accv = fmaf(pw, vc[(size_t)i * dp], accv);
        }
        aLs[(size_t)r * dp + v] = acc * inv_s;
        if (last) ys[(size_t)r * dp + v] = accv * inv_s;
      }
      if (lane == 0) cLs[r] = sz * inv_s - (zmax + logf(s));
      __syncwarp();
    }
    __syncthreads();

    // ---------------------------------------------------------------- L half-step (Eq. 8, 9 / Eq. 4)
    // pair (jj, l): Z_L[k] = scale * <Q(l,j), alpha_L(j,k)> - c_L(j,k); L = softmax_k Z_L
    for (int p = warp; p < nj * m; p += kWarps) {
      const int jj = p / m, l = p - jj * m;
      const float* q = Qs + (size_t)p * dp;
      float zmax = -INFINITY;
      for (int k = lane; k < m; k += 32) {
        const float* al = aLs + (size_t)(jj * m + k) * dp;
        float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
        int v = 0;
        for (; v + 3 < d; v += 4) {
          acc0 = fmaf(q[v], al[v], acc0);
          acc1 = fmaf(q[v + 1], al[v + 1], acc1);
          acc2 = fmaf(q[v + 2], al[v + 2], acc2);
          acc3 = fmaf(q[v + 3], al[v + 3], acc3);
        }
        for (; v < d; ++v) acc0 = fmaf(q[v], al[v], acc0);
        const float z = ((acc0 + acc1) + (acc2 + acc3)) * scale - cLs[jj * m + k];
        zs[k] = z;
        zmax = fmaxf(zmax, z);
      }
      zmax = warp_max(zmax);
      float s = 0.f;
      for (int k = lane; k < m; k += 32) {
        const float pw = expf(zs[k] - zmax);
        zs[k] = pw;
        s += pw;
      }
      s = warp_sum(s);
      __syncwarp();
      const float inv_s = 1.f / s;
      if (last) {
        // log-sum-exp of row b l + j: summed over a head's rows it is the objective (Eq. 6)
        if (row_lse != nullptr && lane == 0) row_lse[(size_t)h * N + (size_t)l * b + j0 + jj] = zmax + logf(s);
        TIn* out = Y + io_off(h, l * b + j0 + jj, N, d, H);
        const float* yc = ys + (size_t)jj * m * dp;
        for (int v = lane; v < d; v += 32) {
          float acc = 0.f;
          for (int k = 0; k < m; ++k) acc = fmaf(zs[k], yc[(size_t)k * dp + v], acc);
          st_from_float(out + v, acc * inv_s);
        }
      } else {
        for (int k = lane; k < m; k += 32) Ls[(size_t)p * mp + k] = zs[k] * inv_s;
      }
      __syncwarp();
    }
    if (!last) {
      __syncthreads();
      // pair (jj, k): alpha_R(k,j) = sum_l L[l,k] Q(l,j) (unscaled Q), c_R(k,j) = sum_l L[l,k]
      for (int p = warp; p < nj * m; p += kWarps) {
        const int jj = p / m, k = p - jj * m;
        const float* lc = Ls + (size_t)jj * m * mp + k;
        const float* qc = Qs + (size_t)jj * m * dp;
        for (int v = lane; v < d; v += 32) {
          float acc = 0.f;
          for (int l = 0; l < m; ++l) acc = fmaf(lc[(size_t)l * mp], qc[(size_t)l * dp + v], acc);
          aRs[(size_t)p * dp + v] = acc;
        }
        float c = 0.f;
        for (int l = lane; l < m; l += 32) c += lc[(size_t)l * mp];
        c = warp_sum(c);
        if (lane == 0) cRs[p] = c;
      }
      __syncthreads();
    }
  }
}

int launch(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int d, int b, int m,
           int T, int dtype, float scale, int n_valid, int H, float* lse, cudaStream_t st);

#ifdef MA_TU_FUSED_F32
template <typename TIn>
inline int launch_t(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int d, int b,
                    int m, int T, float scale, int n_valid, int H, float* lse, cudaStream_t st) {
  static int sms[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 7;
  if (sms[dev] == 0 && cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return 7;
  const int JT = positions_per_cta(N, d, b, m, BH, sms[dev]);
  if (JT < 1 || BH > 65535) return 4;
  auto kern = monarch_fused_f32<TIn>;
  const size_t smem = smem_floats(N, d, b, m, JT) * 4;
  static bool prepared[64] = {};
  if (!prepared[dev]) {      // once per device: the kernel may use all of shared memory
    if (cudaFuncSetAttribute((const void*)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) !=
        cudaSuccess)
      return 7;
    prepared[dev] = true;
  }
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((b + JT - 1) / JT, BH);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, (const TIn*)Q, (const TIn*)K, (const TIn*)V, (TIn*)Y, N, d, b, m, T,
                            scale, n_valid, H, JT, lse) == cudaSuccess
             ? 0
             : 7;
}

int launch(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int d, int b, int m,
           int T, int dtype, float scale, int n_valid, int H, float* lse, cudaStream_t st) {
  if (dtype == 0) return launch_t<float>(Q, K, V, Y, BH, N, d, b, m, T, scale, n_valid, H, lse, st);
  if (dtype == 1) return launch_t<__half>(Q, K, V, Y, BH, N, d, b, m, T, scale, n_valid, H, lse, st);
  return launch_t<__nv_bfloat16>(Q, K, V, Y, BH, N, d, b, m, T, scale, n_valid, H, lse, st);
}
#endif  // MA_TU_FUSED_F32

}  // namespace ffused
}  // namespace ma
