// C-ABI boundary of libmonarch_attn: argument validation, workspace layout, path selection and
// kernel launches.  No torch types; plain device/host pointers and sizes only.
#include "../../include/monarch_attn.h"
#include "../../include/monarch_attn_test.h"

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "generic_kernels.cuh"
#include "tensor_path.cuh"
#include "tensor_persistent.cuh"
#include "tensor_decoupled.cuh"
#include "fused_small.cuh"
#include "fused_f32.cuh"
#include "fused_jsplit.cuh"
#include "tile_mma.cuh"

namespace ma {

static thread_local int g_last_launches = 0;

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int esize(int dtype) { return dtype == MA_F32 ? 4 : 2; }

struct Problem {
  int batch, heads, N, d, b, T, dtype, m, BH;
  int n_valid;   // keys b k + i >= n_valid are masked out (App. C.3); N when there is no padding
  int H;         // 0: [batch][heads][N][d]; heads: [batch][N][heads][d]
  float* lse;    // optional output [batch*heads][N]: row log-sum-exp of the final L half-step
  const int* seq_len;   // optional DEVICE array [batch]: valid length of every sequence (App. C.3)
};

static int validate_shape(int batch, int heads, int N, int d, int b, int T, int dtype, Problem* p) {
  if (dtype != MA_F32 && dtype != MA_F16 && dtype != MA_BF16) return MA_ERR_DTYPE;
  if (batch <= 0 || heads <= 0 || N <= 0 || d <= 0 || b <= 0 || T < 1) return MA_ERR_SHAPE;
  if (N % b != 0) return MA_ERR_SHAPE;
  if ((long long)batch * heads > 0x7fffffffLL / 2) return MA_ERR_SHAPE;
  *p = Problem{batch, heads, N, d, b, T, dtype, N / b, batch * heads, N, 0, nullptr, nullptr};
  return MA_OK;
}

// ------------------------------------------------------------------ generic path
constexpr size_t kStatusBytes = 256;
constexpr size_t kMaxSmem = 227 * 1024;

static bool generic_supported(const Problem& p) {
  if (p.BH > 65535) return false;   // gridDim.y
  size_t r = generic::r_step_smem_floats(p.b, p.d, true) * 4;
  size_t l = generic::l_step_smem_floats(p.m, p.d, false) * 4;
  size_t lf = generic::l_step_smem_floats(p.m, p.d, true) * 4;
  return r <= kMaxSmem && l <= kMaxSmem && lf <= kMaxSmem;
}

struct GenericWs {
  int* status;
  float *aL, *aR, *y, *cL, *cR;
  size_t bytes;
};

static GenericWs generic_layout(const Problem& p, void* base) {
  GenericWs w;
  char* c = (char*)base;
  size_t off = 0;
  size_t big = align_up((size_t)p.BH * p.N * p.d * 4, 256);
  size_t small = align_up((size_t)p.BH * p.N * 4, 256);
  w.status = (int*)(c + off); off += kStatusBytes;
  w.aL = (float*)(c + off); off += big;
  w.aR = (float*)(c + off); off += big;
  w.y = (float*)(c + off); off += big;
  w.cL = (float*)(c + off); off += small;
  w.cR = (float*)(c + off); off += small;
  w.bytes = off;
  return w;
}

// Launch with programmatic stream serialisation (the kernels wait for the launch before them
// themselves: generic::grid_dependency_sync).
template <typename... KArgs, typename... Args>
static cudaError_t launch_serialised(void (*kern)(KArgs...), dim3 grid, int threads, size_t smem,
                                     cudaStream_t st, Args... args) {
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

template <typename TIn>
static int launch_generic_t(const Problem& p, const TIn* Q, const TIn* K, const TIn* V, TIn* Y,
                            float scale, const GenericWs& w, cudaStream_t st) {
  using namespace generic;
  int launches = 0;
  dim3 gr(p.m, p.BH), gl(p.b, p.BH);
  auto set_smem = [](const void* f, size_t bytes) {
    return cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  };
  if (cudaMemsetAsync(w.status, 0, kStatusBytes, st) != cudaSuccess) return MA_ERR_CUDA;
  for (int t = 1; t <= p.T; ++t) {
    const bool first = (t == 1), last = (t == p.T);
    size_t rs = r_step_smem_floats(p.b, p.d, last) * 4;
#define MA_LAUNCH_R(FIRST, WITHV)                                                              \
  do {                                                                                         \
    if (set_smem((const void*)r_step_kernel<TIn, FIRST, WITHV>, rs) != cudaSuccess)            \
      return MA_ERR_CUDA;                                                                      \
    if (launch_serialised(r_step_kernel<TIn, FIRST, WITHV>, gr, kThreads, rs, st, Q, K, V, w.aR, \
                          w.cR, w.aL, w.cL, w.y, p.N, p.d, p.b, p.m, scale, p.n_valid,          \
                          p.H, p.seq_len, p.heads) != cudaSuccess)                              \
      return MA_ERR_CUDA;                                                                       \
  } while (0)
    if (first && last) MA_LAUNCH_R(true, true);
    else if (first) MA_LAUNCH_R(true, false);
    else if (last) MA_LAUNCH_R(false, true);
    else MA_LAUNCH_R(false, false);
#undef MA_LAUNCH_R
    ++launches;
    size_t ls = l_step_smem_floats(p.m, p.d, last) * 4;
    if (last) {
      if (set_smem((const void*)l_step_kernel<TIn, true>, ls) != cudaSuccess) return MA_ERR_CUDA;
      if (launch_serialised(l_step_kernel<TIn, true>, gl, kThreads, ls, st, Q, w.aL, w.cL, w.y, w.aR, w.cR, Y,
                            p.N, p.d, p.b, p.m, scale, p.H, p.lse, p.seq_len, p.heads) != cudaSuccess)
        return MA_ERR_CUDA;
    } else {
      if (set_smem((const void*)l_step_kernel<TIn, false>, ls) != cudaSuccess) return MA_ERR_CUDA;
      if (launch_serialised(l_step_kernel<TIn, false>, gl, kThreads, ls, st, Q, w.aL, w.cL, w.y, w.aR, w.cR, Y,
                            p.N, p.d, p.b, p.m, scale, p.H, (float*)nullptr, p.seq_len, p.heads) != cudaSuccess)
        return MA_ERR_CUDA;
    }
    ++launches;
  }
  if (cudaGetLastError() != cudaSuccess) return MA_ERR_CUDA;
  g_last_launches = launches;
  return MA_OK;
}

static int launch_generic(const Problem& p, const void* Q, const void* K, const void* V, void* Y,
                          float scale, void* ws, cudaStream_t st) {
  GenericWs w = generic_layout(p, ws);
  switch (p.dtype) {
    case MA_F32:
      return launch_generic_t<float>(p, (const float*)Q, (const float*)K, (const float*)V,
                                     (float*)Y, scale, w, st);
    case MA_F16:
      return launch_generic_t<__half>(p, (const __half*)Q, (const __half*)K, (const __half*)V,
                                      (__half*)Y, scale, w, st);
    default:
      return launch_generic_t<__nv_bfloat16>(p, (const __nv_bfloat16*)Q, (const __nv_bfloat16*)K,
                                             (const __nv_bfloat16*)V, (__nv_bfloat16*)Y, scale, w,
                                             st);
  }
}

// ------------------------------------------------------------------ path selection
// `plain`: the call has no mask and no row_lse output (the kernel split by in-block position
// serves nothing else; the entry point for the other layout selects it itself).
static int resolve_path(const Problem& p, int path, bool plain = true) {
  if (path == MA_PATH_AUTO) {
    // From the third round on, plain 16-bit states are too coarse on peaky logits (they are fed
    // back round after round: about one head in 300 of the N = 256 recipe exceeds 1e-2 at T = 3).
    // The fused per-head kernel and the tcgen05 kernels keep such states; the tile kernels switch to
    // hi + lo pairs from T = 3 on, so they take every 16-bit shape they support then.
    // (short sequences with small blocks: the fused per-head kernel with hi + lo states, one launch)
    if (p.T >= 3 && fsmall::supported_hilo(p.N, p.d, p.b, p.m, p.dtype, p.T)) return MA_PATH_FUSED_SMALL;
    if (p.T >= 3 && tile::supported(p.N, p.d, p.b, p.m, p.dtype, p.BH)) return MA_PATH_TILE_MMA;
    // N = 1024 as 32 x 32: one launch, a head split over four CTAs by in-block position
    if (plain && p.T <= 2 && jsplit::supported(p.N, p.d, p.b, p.m, p.dtype, p.BH)) return MA_PATH_FUSED_JSPLIT;
    // Short sequences with small blocks: one CTA per head, states in shared memory.
    if (p.b <= 16 && p.m <= 16 && fsmall::supported(p.N, p.d, p.b, p.m, p.dtype, p.T))
      return MA_PATH_FUSED_SMALL;
    if (tp::supported(p.N, p.d, p.b, p.m, p.dtype, p.BH)) return MA_PATH_TENSOR;
    // (blocks of more than 32 rows: the tile kernels' two launches are as fast or faster with inputs
    // in HBM, measured; the fused kernel takes them when asked for by name, and for the mask entries)
    if (p.b <= 32 && fsmall::supported(p.N, p.d, p.b, p.m, p.dtype, p.T)) return MA_PATH_FUSED_SMALL;
    if (tile::supported(p.N, p.d, p.b, p.m, p.dtype, p.BH)) return MA_PATH_TILE_MMA;
    // fp32 inputs: short sequences in one launch with the states in shared memory
    if (p.dtype == MA_F32 && p.BH <= 65535 && ffused::supported(p.N, p.d, p.b, p.m)) return MA_PATH_FUSED_F32;
    if (generic_supported(p)) return MA_PATH_GENERIC;
    return -1;
  }
  if (path == MA_PATH_GENERIC) return generic_supported(p) ? path : -1;
  if (path == MA_PATH_FUSED_F32) return (p.BH <= 65535 && ffused::supported(p.N, p.d, p.b, p.m)) ? path : -1;
  if (path == MA_PATH_FUSED_JSPLIT)
    return (plain && jsplit::supported(p.N, p.d, p.b, p.m, p.dtype, p.BH)) ? path : -1;
  if (path == MA_PATH_TILE_MMA) return tile::supported(p.N, p.d, p.b, p.m, p.dtype, p.BH) ? path : -1;
  if (path == MA_PATH_FUSED_SMALL)
    return fsmall::supported(p.N, p.d, p.b, p.m, p.dtype, p.T) ? path : -1;
  if (path == MA_PATH_TENSOR) return tp::supported(p.N, p.d, p.b, p.m, p.dtype, p.BH) ? path : -1;
  if (path == MA_PATH_TENSOR_TMEM)
    return (tp::supported(p.N, p.d, p.b, p.m, p.dtype, p.BH) &&
            tp::tmem_kernel_supported(p.b, p.H, p.lse, p.n_valid < p.N ? p.n_valid : 0))
               ? path
               : -1;
  if (path == MA_PATH_TENSOR_BASIC)
    return tensor::supported(p.N, p.d, p.b, p.m, p.dtype, p.BH) ? path : -1;
  return -1;
}

// Path choice of the entry points that only the second-generation tensor kernel, the general fused
// kernel (`with_fused_small`), the warp-MMA tile kernels and the generic kernels serve:
// AUTO, TENSOR, FUSED_SMALL, TILE_MMA or GENERIC; -1 if none applies.
static int resolve_tensor_or_generic(const Problem& p, int path, bool with_fused_small = false) {
  if (path == MA_PATH_AUTO) {
    const int r = resolve_path(p, MA_PATH_AUTO, false);
    if (r != MA_PATH_FUSED_SMALL || with_fused_small) return r;
    if (tile::supported(p.N, p.d, p.b, p.m, p.dtype, p.BH)) return MA_PATH_TILE_MMA;
    return generic_supported(p) ? MA_PATH_GENERIC : -1;
  }
  if (path == MA_PATH_TENSOR || path == MA_PATH_TILE_MMA || path == MA_PATH_GENERIC ||
      path == MA_PATH_FUSED_F32 || (path == MA_PATH_FUSED_SMALL && with_fused_small))
    return resolve_path(p, path, false);
  return -1;
}

static size_t workspace_bytes_for(const Problem& p, int resolved) {
  if (resolved == MA_PATH_GENERIC) return generic_layout(p, nullptr).bytes;
  if (resolved == MA_PATH_FUSED_SMALL || resolved == MA_PATH_FUSED_F32 || resolved == MA_PATH_FUSED_JSPLIT)
    return kStatusBytes;   // no states leave the chip
  if (resolved == MA_PATH_TILE_MMA) return tile::workspace_bytes(p.BH, p.N, p.d, p.T);
  if (resolved == MA_PATH_TENSOR_BASIC) return tensor::workspace_bytes(p.BH, p.N, p.d, p.b, p.T);
  if (resolved == MA_PATH_TENSOR || resolved == MA_PATH_TENSOR_TMEM)
    return tp::workspace_bytes(p.BH, p.N, p.T, tp::uses_hilo(p.dtype, p.b));
  return 0;
}

// ------------------------------------------------------------------ library-owned buffers
constexpr int kMaxDevices = 64;
struct DeviceBuffers {
  void* ws = nullptr;
  size_t ws_bytes = 0;
  long long armed_key = -1;   // problem whose status block / counters the workspace is armed for
  void* stage = nullptr;   // Q, K, V, Y staging for the host entry point
  size_t stage_bytes = 0;
  // host entry point: kernels and the copy back run on streams of their own, so that the compute
  // and the device-to-host copy of one chunk of heads overlap the host-to-device copies of the
  // next (PCIe is full duplex)
  cudaStream_t compute = nullptr, d2h = nullptr;
  cudaEvent_t chunk_in[8] = {}, chunk_done[8] = {};
  cudaEvent_t all_back = nullptr;
};
constexpr int kHostChunks = 8;
static int g_host_chunks = 4;   // chunks a host call is cut into (<= kHostChunks)
static DeviceBuffers g_dev[kMaxDevices];

static int grow(void** ptr, size_t* have, size_t need) {
  if (*have >= need) return MA_OK;
  if (*ptr) {
    if (cudaDeviceSynchronize() != cudaSuccess) return MA_ERR_CUDA;
    cudaFree(*ptr);
    *ptr = nullptr;
    *have = 0;
  }
  size_t sz = align_up(need, (size_t)1 << 20);
  if (cudaMalloc(ptr, sz) != cudaSuccess) {
    cudaGetLastError();
    *ptr = nullptr;
    return MA_ERR_CUDA;
  }
  // the status word starts clear (kernels that never arm the workspace themselves only ever set it)
  if (cudaMemset(*ptr, 0, sz < 256 ? sz : 256) != cudaSuccess) return MA_ERR_CUDA;
  *have = sz;
  return MA_OK;
}

static int fwd_ex(const void* Q, const void* K, const void* V, void* Y, const Problem& p,
                  float scale, int resolved, void* ws, size_t ws_bytes, cudaStream_t st,
                  bool ws_armed = false) {
  if (!ws || ws_bytes < workspace_bytes_for(p, resolved)) return MA_ERR_WORKSPACE;
  if (((uintptr_t)ws & 255) != 0) return MA_ERR_ALIGN;
  if (resolved == MA_PATH_GENERIC) return launch_generic(p, Q, K, V, Y, scale, ws, st);
  if (resolved == MA_PATH_FUSED_SMALL) {
    int rc = fsmall::launch(Q, K, V, Y, p.BH, p.N, p.d, p.b, p.m, p.T, p.dtype, scale, p.n_valid, p.H, p.lse, st,
                            p.seq_len, p.heads);
    if (rc == MA_OK) g_last_launches = 1;
    return rc;
  }
  if (resolved == MA_PATH_FUSED_F32) {
    int rc = ffused::launch(Q, K, V, Y, p.BH, p.N, p.d, p.b, p.m, p.T, p.dtype, scale, p.n_valid, p.H, p.lse, st);
    if (rc == MA_OK) g_last_launches = 1;
    return rc;
  }
  if (resolved == MA_PATH_FUSED_JSPLIT) {
    int rc = jsplit::launch(Q, K, V, Y, p.BH, p.T, p.dtype, scale, (int*)ws, st, p.H);
    if (rc == MA_OK) g_last_launches = 1;
    return rc;
  }
  if (resolved == MA_PATH_TILE_MMA) {
    tile::Args a{Q, K, V, Y, p.lse, p.BH, p.N, p.d, p.b, p.m, p.T, p.n_valid, p.H, scale, p.seq_len, p.heads};
    int n = 0;
    int rc = tile::launch(a, p.dtype, ws, st, &n);
    if (rc == MA_OK) g_last_launches = n;
    return rc;
  }
  int launches = 0;
  int rc;
  if (resolved == MA_PATH_TENSOR_BASIC)
    rc = tensor::launch(Q, K, V, Y, p.BH, p.N, p.d, p.b, p.T, p.dtype, scale, ws, st, &launches);
  else
    rc = tp::launch(Q, K, V, Y, p.BH, p.N, p.b, p.T, p.dtype, scale, ws, st, &launches,
                    resolved == MA_PATH_TENSOR_TMEM ? 1 : 0,
                    ws_armed, p.H, p.lse, p.n_valid < p.N ? p.n_valid : 0);
  if (rc == MA_OK) g_last_launches = launches;
  return rc;
}

static int check_ptrs(const void* Q, const void* K, const void* V, void* Y, const Problem& p) {
  if (!Q || !K || !V || !Y) return MA_ERR_NULL;
  if ((((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)Y) & 15) != 0) return MA_ERR_ALIGN;
  size_t bytes = (size_t)p.BH * p.N * p.d * esize(p.dtype);
  const char* y0 = (const char*)Y;
  const void* in[3] = {Q, K, V};
  for (int i = 0; i < 3; ++i) {
    const char* a = (const char*)in[i];
    if (y0 < a + bytes && a < y0 + bytes) return MA_ERR_ALIGN;
  }
  return MA_OK;
}

}  // namespace ma

using namespace ma;

extern "C" {

size_t monarch_attn_workspace_bytes(int batch, int heads, int N, int d, int b, int T, int dtype,
                                    int path) {
  Problem p;
  if (validate_shape(batch, heads, N, d, b, T, dtype, &p) != MA_OK) return 0;
  int r = resolve_path(p, path);
  if (r < 0) return 0;
  return workspace_bytes_for(p, r);
}

int monarch_attn_fwd_ex(const void* Q, const void* K, const void* V, void* Y, int batch, int heads,
                        int N, int d, int b, int T, int dtype, float softmax_scale, int path,
                        void* workspace, size_t workspace_bytes, void* stream) {
  Problem p;
  int rc = validate_shape(batch, heads, N, d, b, T, dtype, &p);
  if (rc != MA_OK) return rc;
  rc = check_ptrs(Q, K, V, Y, p);
  if (rc != MA_OK) return rc;
  if (!(softmax_scale == softmax_scale) || isinf(softmax_scale)) return MA_ERR_SHAPE;
  int r = resolve_path(p, path);
  if (r < 0) return MA_ERR_UNSUPPORTED;
  return fwd_ex(Q, K, V, Y, p, softmax_scale, r, workspace, workspace_bytes, (cudaStream_t)stream);
}

int monarch_attn_fwd_padded(const void* Q, const void* K, const void* V, void* Y, int batch,
                            int heads, int N, int d, int b, int T, int dtype, float softmax_scale,
                            int n_valid, void* workspace, size_t workspace_bytes, void* stream) {
  Problem p;
  int rc = validate_shape(batch, heads, N, d, b, T, dtype, &p);
  if (rc != MA_OK) return rc;
  // less than one block of padding: every key block keeps at least one valid key
  if (n_valid > N || n_valid <= N - b) return MA_ERR_SHAPE;
  rc = check_ptrs(Q, K, V, Y, p);
  if (rc != MA_OK) return rc;
  if (!(softmax_scale == softmax_scale) || isinf(softmax_scale)) return MA_ERR_SHAPE;
  // fused kernel for short sequences; the second-generation tensor kernel where a tile row owns a
  // whole key block (b = 64, 128: the mask touches the last block's tiles only); else generic
  int r = -1;
  if ((p.T <= 2 && fsmall::supported(p.N, p.d, p.b, p.m, p.dtype, p.T)) ||
      fsmall::supported_hilo(p.N, p.d, p.b, p.m, p.dtype, p.T))
    r = MA_PATH_FUSED_SMALL;
  else if (resolve_path(p, MA_PATH_AUTO, false) == MA_PATH_TENSOR && p.b != 32) r = MA_PATH_TENSOR;
  else if (tile::supported(p.N, p.d, p.b, p.m, p.dtype, p.BH)) r = MA_PATH_TILE_MMA;
  else if (p.dtype == MA_F32 && p.BH <= 65535 && ffused::supported(p.N, p.d, p.b, p.m)) r = MA_PATH_FUSED_F32;
  else if (generic_supported(p)) r = MA_PATH_GENERIC;
  if (r < 0) return MA_ERR_UNSUPPORTED;
  p.n_valid = n_valid;
  return fwd_ex(Q, K, V, Y, p, softmax_scale, r, workspace, workspace_bytes, (cudaStream_t)stream);
}

int monarch_attn_fwd_varlen(const void* Q, const void* K, const void* V, void* Y, int batch,
                            int heads, int N, int d, int b, int T, int dtype, float softmax_scale,
                            const int* seq_len, void* workspace, size_t workspace_bytes,
                            void* stream) {
  Problem p;
  int rc = validate_shape(batch, heads, N, d, b, T, dtype, &p);
  if (rc != MA_OK) return rc;
  rc = check_ptrs(Q, K, V, Y, p);
  if (rc != MA_OK) return rc;
  if (!seq_len) return MA_ERR_NULL;
  if (((uintptr_t)seq_len & 3) != 0) return MA_ERR_ALIGN;
  if (!(softmax_scale == softmax_scale) || isinf(softmax_scale)) return MA_ERR_SHAPE;
  // short 16-bit sequences with up to two rounds: the fused per-head kernel (one launch); other
  // 16-bit shapes: the warp-MMA tile kernels (hi + lo states from the third round on); else the
  // generic kernels
  int r = -1;
  if ((p.T <= 2 && fsmall::supported(p.N, p.d, p.b, p.m, p.dtype, p.T)) ||
      fsmall::supported_hilo(p.N, p.d, p.b, p.m, p.dtype, p.T))
    r = MA_PATH_FUSED_SMALL;
  else if (tile::supported(p.N, p.d, p.b, p.m, p.dtype, p.BH)) r = MA_PATH_TILE_MMA;
  else if (generic_supported(p)) r = MA_PATH_GENERIC;
  if (r < 0) return MA_ERR_UNSUPPORTED;
  p.seq_len = seq_len;
  return fwd_ex(Q, K, V, Y, p, softmax_scale, r, workspace, workspace_bytes, (cudaStream_t)stream);
}

int monarch_attn_fwd_objective(const void* Q, const void* K, const void* V, void* Y, int batch,
                               int heads, int N, int d, int b, int T, int dtype,
                               float softmax_scale, int path, float* row_lse, void* workspace,
                               size_t workspace_bytes, void* stream) {
  Problem p;
  int rc = validate_shape(batch, heads, N, d, b, T, dtype, &p);
  if (rc != MA_OK) return rc;
  rc = check_ptrs(Q, K, V, Y, p);
  if (rc != MA_OK) return rc;
  if (!row_lse) return MA_ERR_NULL;
  if (((uintptr_t)row_lse & 3) != 0) return MA_ERR_ALIGN;
  if (!(softmax_scale == softmax_scale) || isinf(softmax_scale)) return MA_ERR_SHAPE;
  const int r = resolve_tensor_or_generic(p, path, true);
  if (r < 0) return MA_ERR_UNSUPPORTED;
  p.lse = row_lse;
  return fwd_ex(Q, K, V, Y, p, softmax_scale, r, workspace, workspace_bytes, (cudaStream_t)stream);
}

int monarch_attn_fwd_bshd(const void* Q, const void* K, const void* V, void* Y, int batch, int N,
                          int heads, int d, int b, int T, int dtype, float softmax_scale, int path,
                          void* workspace, size_t workspace_bytes, void* stream) {
  Problem p;
  int rc = validate_shape(batch, heads, N, d, b, T, dtype, &p);
  if (rc != MA_OK) return rc;
  rc = check_ptrs(Q, K, V, Y, p);
  if (rc != MA_OK) return rc;
  if (!(softmax_scale == softmax_scale) || isinf(softmax_scale)) return MA_ERR_SHAPE;
  // (the kernel split by in-block position takes this layout too: a head is a column offset of
  // its tensor maps)
  int r;
  if (((path == MA_PATH_AUTO && p.T <= 2) || path == MA_PATH_FUSED_JSPLIT) &&
      jsplit::supported(p.N, p.d, p.b, p.m, p.dtype, p.BH))
    r = MA_PATH_FUSED_JSPLIT;
  else
    r = resolve_tensor_or_generic(p, path, true);
  if (r < 0) return MA_ERR_UNSUPPORTED;
  p.H = heads;
  return fwd_ex(Q, K, V, Y, p, softmax_scale, r, workspace, workspace_bytes, (cudaStream_t)stream);
}

int monarch_attn_fwd(const void* Q, const void* K, const void* V, void* Y, int batch, int heads,
                     int N, int d, int b, int T, int dtype, void* stream) {
  Problem p;
  int rc = validate_shape(batch, heads, N, d, b, T, dtype, &p);
  if (rc != MA_OK) return rc;
  rc = check_ptrs(Q, K, V, Y, p);
  if (rc != MA_OK) return rc;
  int r = resolve_path(p, MA_PATH_AUTO);
  if (r < 0) return MA_ERR_UNSUPPORTED;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MA_ERR_CUDA;
  DeviceBuffers& B = g_dev[dev];
  const size_t had = B.ws_bytes;
  rc = grow(&B.ws, &B.ws_bytes, workspace_bytes_for(p, r));
  if (rc != MA_OK) return rc;
  // The persistent kernel leaves its status block and counters zeroed, so the library's own
  // workspace is cleared only when the problem (hence the layout) changes.
  const long long key = ((long long)r << 56) ^ ((long long)p.T << 48) ^ ((long long)p.BH << 24) ^ p.N;
  const bool armed = (r == MA_PATH_TENSOR) && had == B.ws_bytes && B.armed_key == key;
  rc = fwd_ex(Q, K, V, Y, p, 1.0f / sqrtf((float)d), r, B.ws, B.ws_bytes, (cudaStream_t)stream,
              armed);
  B.armed_key = (rc == MA_OK && r == MA_PATH_TENSOR) ? key : -1;
  return rc;
}

int monarch_attn_fwd_host(const void* Qh, const void* Kh, const void* Vh, void* Yh, int batch,
                          int heads, int N, int d, int b, int T, int dtype, void* stream) {
  Problem p;
  int rc = validate_shape(batch, heads, N, d, b, T, dtype, &p);
  if (rc != MA_OK) return rc;
  if (!Qh || !Kh || !Vh || !Yh) return MA_ERR_NULL;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MA_ERR_CUDA;
  DeviceBuffers& B = g_dev[dev];
  size_t one = align_up((size_t)p.BH * p.N * p.d * esize(p.dtype), 256);
  rc = grow(&B.stage, &B.stage_bytes, 4 * one);
  if (rc != MA_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  char* s = (char*)B.stage;
  if (!B.all_back) {
    if (cudaStreamCreateWithFlags(&B.compute, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&B.d2h, cudaStreamNonBlocking) != cudaSuccess)
      return MA_ERR_CUDA;
    for (int c = 0; c < kHostChunks; ++c)
      if (cudaEventCreateWithFlags(&B.chunk_in[c], cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&B.chunk_done[c], cudaEventDisableTiming) != cudaSuccess)
        return MA_ERR_CUDA;
    if (cudaEventCreateWithFlags(&B.all_back, cudaEventDisableTiming) != cudaSuccess) return MA_ERR_CUDA;
  }
  // (batch, head) units are independent (Sec. 3: every equation is per head), so the call is cut
  // into chunks of units: copy in on `stream`, compute on the library's compute stream, copy back
  // on its copy-back stream, chained by events.
  const size_t unit = (size_t)p.N * p.d * esize(p.dtype);
  const int chunks = (unit % 16 == 0 && p.BH >= g_host_chunks) ? g_host_chunks : 1;
  int launches = 0;
  for (int c = 0; c < chunks; ++c) {
    const int u0 = (int)((long long)p.BH * c / chunks), u1 = (int)((long long)p.BH * (c + 1) / chunks);
    const size_t off = (size_t)u0 * unit, len = (size_t)(u1 - u0) * unit;
    if (cudaMemcpyAsync(s + off, (const char*)Qh + off, len, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(s + one + off, (const char*)Kh + off, len, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(s + 2 * one + off, (const char*)Vh + off, len, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return MA_ERR_CUDA;
    if (cudaEventRecord(B.chunk_in[c], st) != cudaSuccess ||
        cudaStreamWaitEvent(B.compute, B.chunk_in[c], 0) != cudaSuccess)
      return MA_ERR_CUDA;
    rc = monarch_attn_fwd(s + off, s + one + off, s + 2 * one + off, s + 3 * one + off, 1, u1 - u0, N, d, b,
                          T, dtype, (void*)B.compute);
    if (rc != MA_OK) return rc;
    launches += g_last_launches;
    if (cudaEventRecord(B.chunk_done[c], B.compute) != cudaSuccess ||
        cudaStreamWaitEvent(B.d2h, B.chunk_done[c], 0) != cudaSuccess ||
        cudaMemcpyAsync((char*)Yh + off, s + 3 * one + off, len, cudaMemcpyDeviceToHost, B.d2h) != cudaSuccess)
      return MA_ERR_CUDA;
  }
  // the caller's stream is done when the last result is back
  if (cudaEventRecord(B.all_back, B.d2h) != cudaSuccess || cudaStreamWaitEvent(st, B.all_back, 0) != cudaSuccess)
    return MA_ERR_CUDA;
  g_last_launches = launches;
  return MA_OK;
}

int monarch_attn_device_status(const void* workspace, void* stream) {
  const void* ws = workspace;
  if (!ws) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MA_ERR_CUDA;
    ws = g_dev[dev].ws;
    if (!ws) return MA_OK;
  }
  int word = 0;
  if (cudaMemcpyAsync(&word, ws, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream) !=
      cudaSuccess)
    return MA_ERR_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return MA_ERR_CUDA;
  if (word != 0 && !workspace) {   // an aborted run leaves counters behind: clear on the next call
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices) g_dev[dev].armed_key = -1;
  }
  return word == 0 ? MA_OK : MA_ERR_TIMEOUT;
}

int monarch_attn_last_launch_count(void) { return g_last_launches; }

}  // extern "C"

// ------------------------------------------------------------------ no-allocation entry point
// Scratch for monarch_attn_fwd_noalloc lives in the library image.  In host code the name of a
// __device__ array is only a handle for the runtime, never a device address: the address is
// looked up once per device with cudaGetSymbolAddress and that pointer is what kernels receive.
static __device__ __align__(256) unsigned char g_noalloc_scratch[MONARCH_ATTN_NOALLOC_SCRATCH_BYTES];
static void* g_noalloc_ptr[ma::kMaxDevices] = {nullptr};

extern "C" {

int monarch_attn_fwd_noalloc(const void* Q, const void* K, const void* V, void* Y, int batch,
                             int heads, int N, int d, int b, int T, int dtype, void* stream) {
  Problem p;
  int rc = validate_shape(batch, heads, N, d, b, T, dtype, &p);
  if (rc != MA_OK) return rc;
  rc = check_ptrs(Q, K, V, Y, p);
  if (rc != MA_OK) return rc;
  if (!generic_supported(p)) return MA_ERR_UNSUPPORTED;
  if (generic_layout(p, nullptr).bytes > (size_t)MONARCH_ATTN_NOALLOC_SCRATCH_BYTES)
    return MA_ERR_TOO_LARGE;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MA_ERR_CUDA;
  if (!g_noalloc_ptr[dev]) {   // set-up, once per device, with that device current
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return MA_ERR_CUDA;
    }
    g_noalloc_ptr[dev] = ptr;
  }
  return launch_generic(p, Q, K, V, Y, 1.0f / sqrtf((float)d), g_noalloc_ptr[dev],
                        (cudaStream_t)stream);
}

int monarch_attn_debug_knob(int knob, long long value) {
  if (knob == 1) {
    tp::knobs().wait_cycles = value > 0 ? value : tensor::kWaitCycles;
  } else if (knob == 2) {
    tp::knobs().skip_first_half_step = value != 0;
  } else if (knob == 3) {
    g_host_chunks = value < 1 ? 1 : (value > kHostChunks ? kHostChunks : (int)value);
  } else {
    return MA_ERR_SHAPE;
  }
  for (int d = 0; d < kMaxDevices; ++d) g_dev[d].armed_key = -1;
  return MA_OK;
}

int monarch_attn_set_trace_buffer(void* device_buffer, size_t bytes) {
  if (device_buffer != nullptr && bytes < (size_t)4 * 64 * 8 * sizeof(long long)) return MA_ERR_WORKSPACE;
  tp::trace_buffer() = (long long*)device_buffer;
  return MA_OK;
}

const char* monarch_attn_status_string(int status) {
  switch (status) {
    case MA_OK: return "ok";
    case MA_ERR_NULL: return "a required pointer is NULL";
    case MA_ERR_SHAPE: return "invalid shape: need batch, heads, N, d, b > 0, N % b == 0, T >= 1";
    case MA_ERR_DTYPE: return "unknown dtype";
    case MA_ERR_UNSUPPORTED: return "no kernel on the requested path for this (b, m, d, dtype)";
    case MA_ERR_ALIGN: return "pointer not aligned, or output aliases an input";
    case MA_ERR_WORKSPACE: return "workspace missing or too small";
    case MA_ERR_CUDA: return "a CUDA call failed";
    case MA_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case MA_ERR_TOO_LARGE: return "problem exceeds the scratch built into monarch_attn_fwd_noalloc";
    default: return "unknown status";
  }
}

}  // extern "C"
