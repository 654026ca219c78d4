// Shared plumbing of the persistent tensor-core kernels: all 2T half-steps of the forward pass in
// ONE launch.  One CTA per SM walks a static list of 128-row tiles ordered half-step by half-step
// (R1 of every head, L1 of every head, R2 ...).  A tile of half-step p of head h may start once
// every tile of half-step p-1 of the same head has been stored; that is tracked with one counter
// per (half-step, head) in the workspace.  Because the list is ordered and every CTA takes its tiles
// in increasing order, each dependency points to a tile some resident CTA has already taken, so the
// (bounded) waits cannot deadlock as long as every CTA of the grid is resident (grid <= number of
// SMs, one CTA per SM: the kernels need the whole GPU); with the phase-major order a dependency is
// almost a whole half-step old when it is needed and the waits are normally free.
//
// This header holds what the kernels share: the parameter block (tensor maps, state arrays,
// counters), the tile iterator, bounded waits and small PTX wrappers, and the host-side set-up
// (workspace layout, tensor maps cached per problem, launch).  The kernels themselves are in
// tensor_decoupled.cuh (operand rings in shared memory, P through shared memory) and
// tensor_tmem.cuh (P handed to the apply MMA through tensor memory).
#pragma once
#include <mutex>

#include "tensor_path.cuh"

namespace ma {
namespace tp {

using namespace ma::tensor;

constexpr int kSlot = kTileBytes;   // 16 KB

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
  int head_groups;     // the heads are walked in this many groups, each through all its half-steps (power of two)
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
// (tiles_per_head is a power of two on this path).  Order of the tile list: the heads are cut into
// `head_groups` groups; a group goes through all its 2T half-steps (half-step-major inside the
// group) before the next group starts.  Every dependency still points backwards in the list, and
// with a group's inputs and states smaller than L2 the later half-steps find Q and K there instead
// of reading them from HBM again.
struct TileIter {
  int p, local, step, tpg, tph_shift, tph_mask, kTiles, lastR, h0, hpg, phases;
  __device__ __forceinline__ TileIter(const Params& P, int g0, int step_, int kTiles_)
      : step(step_), tpg(P.tiles_per_phase / P.head_groups), kTiles(kTiles_), lastR(2 * P.T - 2),
        hpg(P.BH / P.head_groups), phases(2 * P.T) {
    const int per_group = phases * tpg;
    const int grp = g0 / per_group;
    const int r = g0 - grp * per_group;
    p = r / tpg;
    local = r - p * tpg;
    h0 = grp * hpg;
    tph_shift = 31 - __clz(P.tiles_per_head);
    tph_mask = P.tiles_per_head - 1;
  }
  __device__ __forceinline__ Tile get() const {
    Tile t;
    t.p = p;
    t.h = h0 + (local >> tph_shift);
    t.idx0 = (local & tph_mask) * kTiles;
    t.isR = (p & 1) == 0;
    t.first = p == 0;
    t.withV = p == lastR;
    t.final_ = p == lastR + 1;
    return t;
  }
  __device__ __forceinline__ void next() {
    local += step;
    while (local >= tpg) {
      local -= tpg;
      if (++p == phases) { p = 0; h0 += hpg; }
    }
  }
};

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

// The kernels (explicitly instantiated in translation units of their own).
//   launch_decoupled: tensor_decoupled.cuh, B in {64, 128}, SB in {32, 64, 128}
//   launch_tmem:      tensor_tmem.cuh, SB == B in {64, 128}
template <typename T, int B, int SB>
cudaError_t launch_decoupled(const Params& P, int grid, cudaStream_t st);
template <typename T, int B>
cudaError_t launch_tmem(const Params& P, int grid, cudaStream_t st);

// mode 0: kernel of tensor_decoupled.cuh; mode 1: kernel of tensor_tmem.cuh (m = b in {64, 128},
// plain calls only: no [batch][N][heads][d] layout, no row log-sum-exp, no padding mask).
int launch(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int b, int T,
           int dtype, float scale, void* ws, cudaStream_t st, int* launches, int mode,
           bool ws_armed, int H = 0, float* lse = nullptr, int n_valid = 0);
inline bool tmem_kernel_supported(int b, int H, const float* lse, int n_valid) {
  return (b == 64 || b == 128) && H == 0 && lse == nullptr && n_valid == 0;
}

#ifdef MA_TU_TENSOR_PERSISTENT
// Tensor maps depend only on the addresses and the shape, and encoding the eleven to thirteen of a
// call costs tens of microseconds of host time: the last few problems' maps are kept.
struct MapKey {
  const void *Q, *K, *V, *Y, *ws;
  int BH, N, SB, dtype, H, T;
  bool operator==(const MapKey& o) const {
    return Q == o.Q && K == o.K && V == o.V && Y == o.Y && ws == o.ws && BH == o.BH && N == o.N &&
           SB == o.SB && dtype == o.dtype && H == o.H && T == o.T;
  }
};
struct MapCache {
  static constexpr int kEntries = 8;
  MapKey key[kEntries];
  Params maps[kEntries];
  bool used[kEntries] = {};
  int next = 0;
  std::mutex mu;
};
inline MapCache& map_cache() {
  static MapCache c;
  return c;
}
inline int sm_count() {   // of the current device
  static int sms[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (sms[dev] == 0 &&
      cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    sms[dev] = 0;
  return sms[dev];
}

struct PersistentChain {      // one event per device: the end of the last persistent launch
  std::mutex mu;
  cudaEvent_t ev[64] = {};
  bool rec[64] = {};
  int dev() const {
    int d = 0;
    return (cudaGetDevice(&d) == cudaSuccess && d >= 0 && d < 64) ? d : -1;
  }
  cudaEvent_t event() {
    const int d = dev();
    if (d < 0) return nullptr;
    if (ev[d] == nullptr && cudaEventCreateWithFlags(&ev[d], cudaEventDisableTiming) != cudaSuccess)
      ev[d] = nullptr;
    return ev[d];
  }
  bool recorded() const { const int d = dev(); return d >= 0 && rec[d]; }
  void set_recorded() { const int d = dev(); if (d >= 0) rec[d] = true; }
};
inline PersistentChain& persistent_chain() {
  static PersistentChain c;
  return c;
}

template <typename T, int B, int SB>
inline int launch_t(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int T_steps,
                    int dtype, float scale, void* ws, cudaStream_t st, int* launches, int mode,
                    bool ws_armed, int H, float* lse, int n_valid) {
  if (mode == 1 && (SB != B || !tmem_kernel_supported(SB, H, lse, n_valid))) return 4;
  // the padding mask only where a tile row owns a whole key block
  if (n_valid != 0 && SB != B) return 4;
  const Ws w = ws_layout(ws, BH, N);
  int* counters = (int*)((char*)ws + w.bytes);
  const int m = N / SB;            // = SB on this path
  const uint64_t rows = (uint64_t)BH * N;
  void* aLlo = (char*)counters + counters_bytes(BH, T_steps);   // used when uses_hilo(dtype, SB)
  Params P;
  {
    MapCache& c = map_cache();
    const MapKey key{Q, K, V, Y, ws, BH, N, SB, dtype, H, T_steps};
    std::lock_guard<std::mutex> lock(c.mu);
    int hit = -1;
    for (int i = 0; i < MapCache::kEntries; ++i)
      if (c.used[i] && c.key[i] == key) hit = i;
    if (hit < 0) {
      constexpr uint32_t kBlk = kRows / SB;     // blocks per tile: one box per tile (blocked views)
      bool ok = make_map_rows_io(&P.tmQ, dtype, (void*)Q, rows, H) &&
                make_map_rows_io(&P.tmK, dtype, (void*)K, rows, H) &&
                make_map_rows_io(&P.tmV, dtype, (void*)V, rows, H) &&
                make_map_rows(&P.tmAR, dtype, w.aR, rows) && make_map_rows(&P.tmAL, dtype, w.aL, rows) &&
                make_map_rows(&P.tmY, dtype, w.y, rows) &&
                make_map_blocked_io(&P.tmALs, dtype, w.aL, m, (uint64_t)BH * SB, SB, kBlk, 0) &&
                make_map_blocked_io(&P.tmYs, dtype, w.y, m, (uint64_t)BH * SB, SB, kBlk, 0) &&
                make_map_blocked_io(&P.tmQs, dtype, (void*)Q, SB, (uint64_t)BH * m, SB, kBlk, H) &&
                make_map_blocked_io(&P.tmARs, dtype, w.aR, SB, (uint64_t)BH * m, SB, kBlk, 0) &&
                make_map_blocked_io(&P.tmOut, dtype, Y, SB, (uint64_t)BH * m, SB, kBlk, H);
      if (ok && uses_hilo(dtype, SB))
        ok = make_map_rows(&P.tmALlo, dtype, aLlo, rows) &&
             make_map_blocked_io(&P.tmALlos, dtype, aLlo, m, (uint64_t)BH * SB, SB, kBlk, 0);
      if (!ok) return 7;
      hit = c.next;
      c.next = (c.next + 1) % MapCache::kEntries;
      c.key[hit] = key;
      c.maps[hit] = P;
      c.used[hit] = true;
    } else {
      P = c.maps[hit];
    }
  }
  P.aL = (uint8_t*)w.aL; P.aR = (uint8_t*)w.aR; P.y = (uint8_t*)w.y; P.out = (uint8_t*)Y;
  P.cL = w.cL; P.cR = w.cR; P.status = w.status; P.counters = counters;
  P.trace = trace_buffer();
  P.m = m; P.BH = BH; P.T = T_steps; P.H = H; P.lse = lse; P.n_valid = n_valid;
  P.tiles_per_head = m / (kRows / SB);
  P.tiles_per_phase = BH * P.tiles_per_head;
  // head groups: as many as keep a group's half-step long enough that a tile's dependencies are
  // long done when its turn comes (measured: C5, 1024 tiles of 128 x 128 per group and half-step,
  // same time and 118 MB instead of 217 MB of DRAM traffic; C4, 1024 tiles of two 64 x 64 blocks,
  // 3 % slower, hence the higher bar for the faster small tiles)
  const int min_tiles = B == 128 ? 1024 : 2048;
  P.head_groups = 1;
  while (BH % (2 * P.head_groups) == 0 && P.tiles_per_phase / (2 * P.head_groups) >= min_tiles) P.head_groups *= 2;
  P.scale = scale;
  P.n_counters = 2 * T_steps * BH;
  P.wait_cycles = knobs().wait_cycles;
  if (!ws_armed) {   // status block and counters start at zero; the kernel leaves them that way
    if (cudaMemsetAsync(ws, 0, kWsStatusBytes, st) != cudaSuccess) return 7;
    if (cudaMemsetAsync(counters, 0, counters_bytes(BH, T_steps), st) != cudaSuccess) return 7;
  }
  const int num_sms = sm_count();
  if (num_sms <= 0) return 7;
  // The grid only makes progress if every CTA is resident (tiles are dealt out statically and wait
  // on each other's results), i.e. if it has the GPU to itself.  Two such launches on different
  // streams could split the SMs between them and starve each other, so launches of this family are
  // chained per device with an event: a later one starts when the earlier one has finished,
  // whatever streams they are on.
  PersistentChain& chain = persistent_chain();
  std::lock_guard<std::mutex> chain_lock(chain.mu);
  cudaEvent_t ev = chain.event();
  if (ev == nullptr) return 7;
  if (chain.recorded() && cudaStreamWaitEvent(st, ev, 0) != cudaSuccess) return 7;
  const int total = 2 * T_steps * P.tiles_per_phase;
  // one launch, dependencies tracked by counters
  P.g_begin = knobs().skip_first_half_step ? P.tiles_per_phase : 0; P.g_end = total; P.check_deps = 1;
  const int grid = total < num_sms ? total : num_sms;
  cudaError_t e;
  if constexpr (SB == B) {
    e = mode == 1 ? launch_tmem<T, B>(P, grid, st) : launch_decoupled<T, B, SB>(P, grid, st);
  } else {
    e = launch_decoupled<T, B, SB>(P, grid, st);
  }
  if (e != cudaSuccess) return 7;
  if (cudaEventRecord(ev, st) != cudaSuccess) return 7;
  chain.set_recorded();
  *launches = 1;
  return 0;
}

int launch(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int b, int T,
           int dtype, float scale, void* ws, cudaStream_t st, int* launches, int mode,
           bool ws_armed, int H, float* lse, int n_valid) {
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
#endif  // MA_TU_TENSOR_PERSISTENT

}  // namespace tp
}  // namespace ma
