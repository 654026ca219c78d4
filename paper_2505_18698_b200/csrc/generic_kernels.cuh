// Generic fp32 SIMT kernels for the MonarchAttention half-steps.
//
// One CTA per tile, one warp per score row.  States (alpha_L, alpha_R, y, c_L, c_R of Sec. 3
// 'Implementation') are fp32 in the workspace.  Any input dtype and any N = m*b whose tile fits
// shared memory.  This is the reference-accuracy CUDA path (fp32 inputs are held to 1e-5) and the
// fallback for shapes the tensor-core path does not cover.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

namespace ma {
namespace generic {

__device__ __forceinline__ float ld_as_float(const float* p) { return *p; }
__device__ __forceinline__ float ld_as_float(const __half* p) { return __half2float(*p); }
__device__ __forceinline__ float ld_as_float(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void st_from_float(float* p, float v) { *p = v; }
__device__ __forceinline__ void st_from_float(__half* p, float v) { *p = __float2half_rn(v); }
__device__ __forceinline__ void st_from_float(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// The half-step kernels are launched with programmatic stream serialisation: the next launch's
// CTAs may take SM slots while this launch's last CTAs drain, but they touch no memory before every
// CTA of the launch before them has finished.
__device__ __forceinline__ void grid_dependency_sync() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

// Shared-memory floats needed by the two kernels (host uses the same formulas).
__host__ __device__ inline size_t r_step_smem_floats(int b, int d, bool with_v) {
  return (size_t)b * (d + 1) * (with_v ? 2 : 1) + (size_t)kWarps * (b + d);
}
__host__ __device__ inline size_t l_step_smem_floats(int m, int d, bool final_step) {
  size_t tiles = (size_t)m * (d + 1) * 2;                       // alpha_L[j], Qb[j]
  size_t extra = final_step ? (size_t)m * (d + 1) : (size_t)m * (m + 1);   // y[j] or L tile
  return tiles + extra + m + (size_t)kWarps * (m + d);
}

// R half-step for key block k of head h (Eq. 7, 9 -> Eq. 10):
//   Z_R[j,i] = scale * <aR[k,j,:], K[b k + i,:]> / cR[k,j];  R = softmax_i Z_R
//   aL[j,k,:] = sum_i R[j,i] K[b k + i,:];  cL[j,k] = sum_i R log R;  (final) y[j,k,:] = sum_i R V
// Element offset of row n of head h (flat index batch * heads + head) in Q, K, V, Y.
// H = 0: [batch][heads][N][d].  H = heads > 0: [batch][N][heads][d].
__device__ __forceinline__ size_t io_off(int h, int n, int N, int d, int H) {
  if (H == 0) return ((size_t)h * N + n) * d;
  return (((size_t)(h / H) * N + n) * H + (h % H)) * d;
}

// FIRST: aR = Q rows b k + j and cR = 1 (L^(0) = identity).
template <typename TIn, bool FIRST, bool WITH_V>
__global__ void __launch_bounds__(kThreads)
r_step_kernel(const TIn* __restrict__ Q, const TIn* __restrict__ K, const TIn* __restrict__ V,
              const float* __restrict__ aR, const float* __restrict__ cR,
              float* __restrict__ aL, float* __restrict__ cL, float* __restrict__ y,
              int N, int d, int b, int m, float scale, int n_valid, int H,
              const int* __restrict__ seq_len, int heads) {
  extern __shared__ float smem[];
  grid_dependency_sync();
  const int k = blockIdx.x, h = blockIdx.y;
  const int dp = d + 1;
  // Batched sequences of different lengths (App. C.3): n_valid is per batch entry.  A key block that
  // lies wholly in the padding is absent from its sequence's problem: alpha_L = y = 0 and
  // c_L = +inf, so that Z_L = -inf and the block gets no weight in the L half-step.
  if (seq_len != nullptr) {
    n_valid = min(max(seq_len[h / heads], 1), N);
    if (k * b >= n_valid) {
      const size_t head_off0 = (size_t)h * N * d;
      for (int e = threadIdx.x; e < b * d; e += kThreads) {
        const int j = e / d, v = e - j * d;
        const size_t row = head_off0 + ((size_t)j * m + k) * d;
        aL[row + v] = 0.f;
        if (WITH_V) y[row + v] = 0.f;
      }
      for (int j = threadIdx.x; j < b; j += kThreads) cL[(size_t)h * N + (size_t)j * m + k] = INFINITY;
      return;
    }
  }
  float* Ks = smem;                                  // [b][d+1]
  float* Vs = Ks + (size_t)b * dp;                   // [b][d+1] if WITH_V
  float* wbuf = Vs + (WITH_V ? (size_t)b * dp : 0);  // per warp: z[b], a[d]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* zs = wbuf + (size_t)warp * (b + d);
  float* as = zs + b;

  const size_t head_off = (size_t)h * N * d;
  for (int e = threadIdx.x; e < b * d; e += kThreads) {
    int i = e / d, v = e - i * d;
    const size_t off = io_off(h, k * b + i, N, d, H) + v;
    Ks[i * dp + v] = ld_as_float(K + off);
    if (WITH_V) Vs[i * dp + v] = ld_as_float(V + off);
  }
  __syncthreads();

  for (int j = warp; j < b; j += kWarps) {
    float inv_c = 1.f;
    if (FIRST) {
      const TIn* q = Q + io_off(h, k * b + j, N, d, H);
      for (int v = lane; v < d; v += 32) as[v] = ld_as_float(q + v);
    } else {
      const float* a = aR + head_off + ((size_t)k * b + j) * d;
      for (int v = lane; v < d; v += 32) as[v] = a[v];
      const float c = cR[(size_t)h * N + (size_t)k * b + j];
      inv_c = c > 1e-30f ? 1.f / c : 0.f;   // c_R underflow: uniform row (Z_R = 0)
    }
    __syncwarp();
    const float f = scale * inv_c;
    float zmax = -INFINITY;
    for (int i = lane; i < b; i += 32) {
      float acc = 0.f;
      const float* kr = Ks + i * dp;
      for (int v = 0; v < d; ++v) acc = fmaf(as[v], kr[v], acc);
      // padding mask (App. C.3, post-padding): key columns b k + i >= n_valid get -inf
      float z = (k * b + i < n_valid) ? acc * f : -INFINITY;
      zs[i] = z;
      zmax = fmaxf(zmax, z);
    }
    zmax = warp_max(zmax);
    float s = 0.f, sz = 0.f;
    for (int i = lane; i < b; i += 32) {
      float z = zs[i];
      const bool valid = z > -INFINITY;
      float p = valid ? expf(z - zmax) : 0.f;
      zs[i] = p;
      s += p;
      if (valid) sz = fmaf(p, z, sz);            // 0 log 0 = 0 for masked keys
    }
    s = warp_sum(s);
    sz = warp_sum(sz);
    __syncwarp();
    const float inv_s = 1.f / s;
    const size_t row = head_off + ((size_t)j * m + k) * d;       // [j][k][:]
    for (int v = lane; v < d; v += 32) {
      float acc = 0.f, accv = 0.f;
      for (int i = 0; i < b; ++i) {
        float p = zs[i];
        acc = fmaf(p, Ks[i * dp + v], acc);
        if (WITH_V) accv = fmaf(p, Vs[i * dp + v], accv);
      }
      aL[row + v] = acc * inv_s;
      if (WITH_V) y[row + v] = accv * inv_s;
    }
    if (lane == 0) cL[(size_t)h * N + (size_t)j * m + k] = sz * inv_s - (zmax + logf(s));
    __syncwarp();
  }
}

// L half-step for in-block position j of head h (Eq. 8, 10 -> Eq. 9 or Eq. 4):
//   Z_L[l,k] = scale * <Q[b l + j,:], aL[j,k,:]> - cL[j,k];  L[j,k,l] = softmax_k Z_L
//   not final: aR[k,j,:] = sum_l L[j,k,l] Q[b l + j,:] (unscaled Q), cR[k,j] = sum_l L[j,k,l]
//   final:     Y[b l + j,:] = sum_k L[j,k,l] y[j,k,:]
template <typename TIn, bool FINAL>
__global__ void __launch_bounds__(kThreads)
l_step_kernel(const TIn* __restrict__ Q, const float* __restrict__ aL, const float* __restrict__ cL,
              const float* __restrict__ y, float* __restrict__ aR, float* __restrict__ cR,
              TIn* __restrict__ Y, int N, int d, int b, int m, float scale, int H,
              float* __restrict__ row_lse, const int* __restrict__ seq_len, int heads) {
  extern __shared__ float smem[];
  grid_dependency_sync();
  const int j = blockIdx.x, h = blockIdx.y;
  // blocks from m_live on lie wholly in the padding of this sequence (App. C.3, batched lengths):
  // as key blocks they carry c_L = +inf (no weight), as query blocks they are left out of the sums
  // over l of Eq. 9 and their rows of Y are zero; their rows of Q are never read
  const int m_live = seq_len != nullptr ? (min(max(seq_len[h / heads], 1), N) + b - 1) / b : m;
  const int dp = d + 1, mp = m + 1;
  float* As = smem;                                  // aL[j]: [m][d+1]
  float* Qs = As + (size_t)m * dp;                   // Qb[j]: [m][d+1]
  float* Xs = Qs + (size_t)m * dp;                   // FINAL: y[j] [m][d+1]; else L tile [m(l)][m+1]
  float* cs = Xs + (FINAL ? (size_t)m * dp : (size_t)m * mp);   // cL[j,:]
  float* wbuf = cs + m;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* ps = wbuf + (size_t)warp * (m + d);

  const size_t head_off = (size_t)h * N * d;
  const float* aLj = aL + head_off + (size_t)j * m * d;
  const float* yj = y + head_off + (size_t)j * m * d;
  for (int e = threadIdx.x; e < m * d; e += kThreads) {
    int r = e / d, v = e - r * d;
    As[r * dp + v] = aLj[e];
    Qs[r * dp + v] = r < m_live ? ld_as_float(Q + io_off(h, r * b + j, N, d, H) + v) : 0.f;
    if (FINAL) Xs[r * dp + v] = yj[e];
  }
  for (int k = threadIdx.x; k < m; k += kThreads) cs[k] = cL[(size_t)h * N + (size_t)j * m + k];
  __syncthreads();

  for (int l = warp; l < m; l += kWarps) {
    if (l >= m_live) {                            // absent query block
      if (FINAL) {
        TIn* out = Y + io_off(h, l * b + j, N, d, H);
        for (int v = lane; v < d; v += 32) st_from_float(out + v, 0.f);
        if (row_lse != nullptr && lane == 0) row_lse[(size_t)h * N + (size_t)l * b + j] = 0.f;
      } else {
        for (int k = lane; k < m; k += 32) Xs[l * mp + k] = 0.f;
      }
      continue;
    }
    const float* q = Qs + l * dp;
    float zmax = -INFINITY;
    for (int k = lane; k < m; k += 32) {
      float acc = 0.f;
      const float* a = As + k * dp;
      for (int v = 0; v < d; ++v) acc = fmaf(q[v], a[v], acc);
      float z = acc * scale - cs[k];
      ps[k] = z;
      zmax = fmaxf(zmax, z);
    }
    zmax = warp_max(zmax);
    float s = 0.f;
    for (int k = lane; k < m; k += 32) {
      float p = expf(ps[k] - zmax);
      ps[k] = p;
      s += p;
    }
    s = warp_sum(s);
    __syncwarp();
    const float inv_s = 1.f / s;
    if (FINAL) {
      // log-sum-exp of row b l + j: summed over a head's rows it is the objective (Eq. 6)
      if (row_lse != nullptr && lane == 0) row_lse[(size_t)h * N + (size_t)l * b + j] = zmax + logf(s);
      TIn* out = Y + io_off(h, l * b + j, N, d, H);
      for (int v = lane; v < d; v += 32) {
        float acc = 0.f;
        for (int k = 0; k < m; ++k) acc = fmaf(ps[k], Xs[k * dp + v], acc);
        st_from_float(out + v, acc * inv_s);
      }
    } else {
      for (int k = lane; k < m; k += 32) Xs[l * mp + k] = ps[k] * inv_s;
    }
    __syncwarp();
  }
  if (!FINAL) {
    __syncthreads();
    for (int k = warp; k < m; k += kWarps) {
      const size_t row = head_off + ((size_t)k * b + j) * d;     // [k][j][:]
      for (int v = lane; v < d; v += 32) {
        float acc = 0.f;
        for (int l = 0; l < m; ++l) acc = fmaf(Xs[l * mp + k], Qs[l * dp + v], acc);
        aR[row + v] = acc;
      }
      float c = 0.f;
      for (int l = lane; l < m; l += 32) c += Xs[l * mp + k];
      c = warp_sum(c);
      if (lane == 0) cR[(size_t)h * N + (size_t)k * b + j] = c;
    }
  }
}

}  // namespace generic
}  // namespace ma
