// Fused per-head kernel for short sequences of any block shape: N = m*b with m <= 32, b <= 64,
// d <= 64 (a multiple of 8), f16/bf16, optional key padding mask (App. C.3) and either layout.
//
// One CTA (8 warps) per (batch, head), one launch for all T rounds.  Q, K, V are read from HBM
// once, the states alpha_L, alpha_R, y, c_L (Sec. 3 'Implementation') never leave shared memory,
// Y is written once.  It covers the shapes whose blocks do not fill a 64-row tensor-core tile:
// N = 256 as 16 blocks of 16, N = 210 as 15 blocks of 14 with 197 valid keys, N = 384 as 16 blocks
// of 24.
//
// Layout.  Every tile (Q, K, V and the states) is stored with the SAME row order, row = k*b + i
// for block k and in-block position i, 128 bytes per row (d padded with zeros to 64).  The
// permutation between the two half-steps (Eq. 9, 10) is therefore only a choice of operand rows:
// an R half-step reads the b consecutive rows of block k, an L half-step reads the m rows (l, j)
// that sit b rows apart.  16-byte chunks are XOR-swizzled with (i & 7) ^ (k & 7), which makes
// 8-row fragment loads conflict-free in both directions.  A warp owns block k (R) or position j
// (L) entirely, so inside a half-step no two warps touch the same rows and the outputs can take
// the place of dead inputs: on the last round alpha_L goes over K, y over V, Y over Q.
//
// Contractions are warp-level mma.sync m16n8k16 in f16 (bf16 inputs are converted to f16 on the way
// in: exact for magnitudes in [6.1e-5, 65504], clamped beyond; the dominant error of a 16-bit
// pipeline is the rounding of alpha_L, and f16 carries three more mantissa bits than bf16).  Blocks are padded to 16 or 32 rows/columns in registers only:
// operand rows past the block are clamped to its last row (finite values), score columns past the
// block or past n_valid get -inf, weight rows past the block are zeroed before a transposed
// product, and output rows past the block are not stored.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "warp_mma.cuh"

namespace ma {
namespace fsmall {

using warpmma::Mma;
using warpmma::col_sum;
using warpmma::ex2;
using warpmma::kLn2;
using warpmma::kLog2e;
using warpmma::ldsm_x2_trans;
using warpmma::ldsm_x4;
using warpmma::ldsm_x4_trans;
using warpmma::lg2;
using warpmma::movm_trans;
using warpmma::quad_max;
using warpmma::quad_sum;

constexpr int kThreads = 256, kWarps = 8, kRowBytes = 128, kMaxSmem = 227 * 1024;
// where stmatrix rows past the end of a block go: 16 bytes per thread
inline size_t dump_bytes(int threads) { return (size_t)threads * 16; }

// Four 8x8 16-bit matrices from accumulator-layout registers; lane L gives the address of row L & 7
// of matrix L >> 3.
__device__ __forceinline__ void stsm_x4(uint32_t saddr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1,%2,%3,%4};" ::"r"(saddr), "r"(r0),
               "r"(r1), "r"(r2), "r"(r3)
               : "memory");
}

// x rounded to f16 (hi) and the f16 rounding of what is left (lo): hi + lo carries 22 bits of x.
template <bool HILO>
__device__ __forceinline__ void split_hilo(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  hi = Mma<__half>::pack(x0, x1);
  lo = 0u;
  if (HILO) {
    const float2 h = Mma<__half>::unpack(hi);
    lo = Mma<__half>::pack(x0 - h.x, x1 - h.y);
  }
}

// Tile layouts.  KS = number of 16-column steps a row holds (4: d <= 64, 5: d <= 80, 8: d <= 128).
// KS = 4: 128-byte rows, row k*b + i, 16-byte chunks XOR-swizzled with (i & 7) ^ (k & 7).
// KS > 4: rows of 32 KS + 16 bytes and 16 more bytes after every block, no swizzle: eight rows of
// a block are 16 bytes (mod 128) apart, and so are the rows (l, j) of eight consecutive blocks, so
// fragment loads are conflict-free in both directions here too.
template <int KS> __device__ __forceinline__ constexpr int row_bytes() { return KS == 4 ? 128 : 32 * KS + 16; }
template <int KS> __host__ __device__ __forceinline__ int block_bytes(int b) {
  return KS == 4 ? b * 128 : b * (32 * KS + 16) + 16;
}
// Byte offset of element (block k, position i, column col) in a tile.
template <int KS> __device__ __forceinline__ uint32_t at(int k, int i, int b, int col) {
  if (KS == 4) {
    const int chunk = (col >> 3) ^ (i & 7) ^ (k & 7);
    return (uint32_t)((k * b + i) * kRowBytes + (chunk << 4) + ((col & 7) << 1));
  }
  return (uint32_t)(k * block_bytes<KS>(b) + i * row_bytes<KS>() + (col << 1));
}

// The same for the 16-column step `step` when the lane's chunk within the step is c (0 or 1):
// stp(rowx(k, i, b, c), step), valid on top of any 128-byte aligned tile address -- one XOR (or
// add) per fragment load instead of the whole index computation.
template <int KS> __device__ __forceinline__ uint32_t rowx(int k, int i, int b, int c) {
  if (KS == 4) return (uint32_t)((k * b + i) * kRowBytes + ((c ^ (i & 7) ^ (k & 7)) << 4));
  return (uint32_t)(k * block_bytes<KS>(b) + i * row_bytes<KS>() + (c << 4));
}
template <int KS> __device__ __forceinline__ uint32_t stp(uint32_t addr, int step) {
  return KS == 4 ? addr ^ (uint32_t)(step << 5) : addr + (uint32_t)(step << 5);
}

inline size_t tile_bytes(int N, int b, int ks) {
  const int m = (N + b - 1) / b;
  return ks == 4 ? (size_t)N * kRowBytes : (size_t)m * ((size_t)b * (32 * ks + 16) + 16);
}
inline int ksteps_for(int d) { return d <= 64 ? 4 : (d <= 80 ? 5 : 8); }
inline size_t smem_bytes(int N, int T, int threads = kThreads, int b = 16, int ks = 4, bool hilo = false) {
  // (alignment slack: the XOR-swizzled layout needs a 1024-byte aligned base, the padded one 128)
  return (size_t)(T == 1 ? 3 : (hilo ? 5 : 4)) * tile_bytes(N, b, ks) + (((size_t)N * 4 + 15) & ~(size_t)15) + dump_bytes(threads) +
         (ks == 4 ? 1024 : 128);
}

// BP: b rounded up to 16, 32, 48 or 64; MP: m rounded up to 16 or 32.  EXACT: b = BP, m = MP, d = 64
// and no mask, known at compile time: every clamp, mask and bounds predicate below folds away and
// the index products become shifts (the instruction stream, not a pipe, bounds this kernel).
// HILO: alpha_L, alpha_R and the weights that feed them are hi + lo pairs of f16 (two more tiles): what
// three or more rounds on peaky logits need (plain 16-bit states, fed back round after round, lose
// 1e-2 on about one head in 300 at T = 3).
template <typename TIn, int BP, int MP, bool EXACT = false, int KS = 4, bool HILO = false>
__global__ void __launch_bounds__((KS == 4 && !HILO && BP <= 32 && (BP == 16 || MP == 16)) ? 2 * kThreads : kThreads, 1)
monarch_fused_small(const TIn* __restrict__ Q, const TIn* __restrict__ K, const TIn* __restrict__ V,
                    TIn* __restrict__ Y, int N, int d, int b, int m, int T_steps, float scale,
                    int n_valid, int H, float* __restrict__ lse, const int* __restrict__ seq_len,
                    int heads) {
  typedef __half T;
  extern __shared__ uint8_t smem_raw[];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // Batched sequences of different lengths (App. C.3): blocks that lie wholly in a sequence's
  // padding are absent from its problem, which is then exactly the problem with
  // m = ceil(length / b) blocks and the appendix's mask in the last of them.  Rows are addressed
  // by (block, position) with the block size b only, so running the smaller problem is a matter
  // of the block count; the rows of Y past it are zeroed, the rows of Q, K, V past it never read.
  if (EXACT) {
    b = BP;
    m = MP;
    N = BP * MP;
    d = 64;
    n_valid = 0x7fffffff;
  }
  const int m_alloc = m;
  if (!EXACT && seq_len != nullptr) {
    n_valid = min(max(seq_len[blockIdx.x / heads], 1), N);
    m = (n_valid + b - 1) / b;
  }
  constexpr uintptr_t kAlign = KS == 4 ? 1024 : 128;
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + kAlign - 1) & ~(kAlign - 1));
  const int tile = KS == 4 ? N * kRowBytes : (N / b) * block_bytes<KS>(b);
  uint8_t* sQ = smem;
  // then K, then V (loaded when the last round starts) ...
  //                                                  ... alpha_L of the earlier rounds until then;
  // alpha_R (T > 1 only) follows it
  // hi + lo states (HILO): Q, K, V, then ONE state tile and its low halves -- alpha_R and alpha_L
  // replace each other in place there (an R tile reads the rows (k, .) it then overwrites, an L tile
  // the rows (., j)), and V has a tile of its own from the start
  float* sCL = reinterpret_cast<float*>(smem + (T_steps == 1 ? 3 : (HILO ? 5 : 4)) * (size_t)tile);   // [k*b + j]
  const uint32_t sQ_u = (uint32_t)__cvta_generic_to_shared(sQ);
  // stmatrix writes whole 8-row matrices: rows past a block's end land in a per-lane dump slot
  const uint32_t dump_u =
      (uint32_t)__cvta_generic_to_shared(reinterpret_cast<uint8_t*>(sCL) + (((size_t)N * 4 + 15) & ~(size_t)15)) +
      threadIdx.x * 16;   // 16-byte aligned like every stmatrix row
  const int st_row = (threadIdx.x & 7) + ((threadIdx.x >> 3) & 1) * 8;   // row within a 16-row tile
  const int st_nt = (threadIdx.x >> 4) & 1;                              // which of a pair of 8-column tiles
  const uint32_t sK_u = sQ_u + tile, sV_u = sK_u + tile;
  const uint32_t sS_u = sQ_u + 3 * tile, sALlo_u = sQ_u + 4 * tile, sARlo_u = sALlo_u;   // HILO only
  const bool v_early = HILO || T_steps == 1;      // V comes in with the first round's loads

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nw = blockDim.x >> 5;    // 8 warps, or 16 where only one CTA fits an SM (16 x 16 blocks)
  const int g = lane >> 2, t = lane & 3;
  const int h_idx = blockIdx.x;
  // Contractions over d always run over the 16 KS padded columns (zeros beyond d: the inputs are
  // zero-filled on the way in and the states are products with them), so every loop unrolls.
  constexpr int ksteps = KS;
  constexpr int LPR = KS == 4 ? 8 : 16;      // lanes that share a row in the copy loops
  constexpr int RPI = 32 / LPR;              // rows per iteration of a warp

  // Rows of this head in global memory.
  const size_t head_base = H == 0 ? (size_t)h_idx * N * d : ((size_t)(h_idx / H) * N * H + (h_idx % H)) * d;
  const size_t row_stride = H == 0 ? (size_t)d : (size_t)H * d;

  // ---- loads.  A warp copies the blocks it owns in the first R half-step itself (Q, K and, when
  // there is one round, V of block k = warp, warp + 8, ...), one asynchronous group per block, and
  // starts on a block as soon as that group has landed: no CTA-wide wait before the first tile.
  // The raw 16-bit values are copied; bf16 is converted to f16 in place by the lane that copied it.
  auto load_block = [&](const TIn* __restrict__ src, int a, int k) {
    const int ch = lane & (LPR - 1);
    if (ch >= 2 * KS) return;
    for (int i = lane / LPR; i < b; i += RPI) {
      const uint32_t off = (uint32_t)(a * tile) + at<KS>(k, i, b, ch * 8);
      if (ch * 8 < d) {
        const TIn* gp = src + head_base + (size_t)(k * b + i) * row_stride + ch * 8;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sQ_u + off), "l"(gp) : "memory");
      } else {
        *reinterpret_cast<uint4*>(smem + off) = make_uint4(0u, 0u, 0u, 0u);   // columns d .. 16 KS - 1
      }
    }
  };
  auto convert_block = [&](int a, int k) {
    if (!Mma<TIn>::is_f16) {
      const int ch = lane & (LPR - 1);
      for (int i = lane / LPR; i < b; i += RPI) {
        if (ch * 8 >= d) continue;
        uint4* p = reinterpret_cast<uint4*>(smem + (size_t)a * tile + at<KS>(k, i, b, ch * 8));
        *p = warpmma::to_f16x8(*p, (const TIn*)nullptr);
      }
    }
  };
  auto wait_pending = [&](int n) {   // until at most n of this thread's copy groups are in flight
    if (n <= 0) asm volatile("cp.async.wait_group 0;" ::: "memory");
    else if (n == 1) asm volatile("cp.async.wait_group 1;" ::: "memory");
    else if (n == 2) asm volatile("cp.async.wait_group 2;" ::: "memory");
    else asm volatile("cp.async.wait_group 3;" ::: "memory");
  };
  int my_tiles = 0;                  // blocks this warp owns in an R half-step (at most 4)
  for (int k = warp; k < m; k += nw) {
    load_block(Q, 0, k);
    load_block(K, 1, k);
    if (v_early) load_block(V, 2, k);
    asm volatile("cp.async.commit_group;" ::: "memory");
    ++my_tiles;
  }

  const float fl = scale * kLog2e;
  for (int step = 1; step <= T_steps; ++step) {
    const bool first = step == 1, last = step == T_steps;
    if (last && !first && !v_early) {   // alpha_L of the round before is dead: V takes its buffer
      for (int k = warp; k < m; k += nw) {
        load_block(V, 2, k);
        asm volatile("cp.async.commit_group;" ::: "memory");
      }
    }
    // ================================================================ R half-step (Eq. 7, 9, 10)
    // tile k: Z_R[j,i] = fl * <alpha_R(k,j), K(k,i)>, softmax over i, alpha_L(k,j) = sum_i R K(k,i)
    {
      const uint32_t sA_u = first ? sQ_u : (HILO ? sS_u : sV_u + tile);   // alpha_R (= Q rows while L is the identity)
      int it = 0;
      for (int k = warp; k < m; k += nw, ++it) {
        if (first || (last && !v_early)) {          // block k may still be on its way
          wait_pending(my_tiles - 1 - it);
          if (first) {
            convert_block(0, k);
            convert_block(1, k);
          }
          if (first ? v_early : true) convert_block(2, k);
          __syncwarp();
        }
        // phase 1: scores and softmax of every 16-row tile of the block; the weights stay in
        // registers as A fragments
        uint32_t pa[BP / 16][BP / 16][4], pal[HILO ? BP / 16 : 1][HILO ? BP / 16 : 1][4];
        float inv_s[BP / 16][2];
#pragma unroll
        for (int rt = 0; rt < BP / 16; ++rt) {
          const int j0 = 16 * rt;
          if (j0 >= b) continue;
          float s[BP / 8][4];
#pragma unroll
          for (int nt = 0; nt < BP / 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) s[nt][e] = 0.f;
          const uint32_t a_u =
              sA_u + rowx<KS>(k, min(j0 + (lane & 7) + ((lane >> 3) & 1) * 8, b - 1), b, lane >> 4);
          uint32_t b_u[BP / 16];
#pragma unroll
          for (int cp = 0; cp < BP / 16; ++cp)
            b_u[cp] = sK_u + rowx<KS>(k, min(16 * cp + (lane & 7) + (lane >> 4) * 8, b - 1), b, (lane >> 3) & 1);
#pragma unroll
          for (int ks = 0; ks < ksteps; ++ks) {
            uint32_t a[4], al[4];
            ldsm_x4(a, stp<KS>(a_u, ks));
            if (HILO && !first) ldsm_x4(al, stp<KS>(a_u - sA_u + sARlo_u, ks));
#pragma unroll
            for (int cp = 0; cp < BP / 16; ++cp) {
              uint32_t bf[4];
              ldsm_x4(bf, stp<KS>(b_u[cp], ks));
              Mma<T>::run(s[2 * cp], a, bf);
              Mma<T>::run(s[2 * cp + 1], a, bf + 2);
              if (HILO && !first) {      // + <alpha_R lo, K>
                Mma<T>::run(s[2 * cp], al, bf);
                Mma<T>::run(s[2 * cp + 1], al, bf + 2);
              }
            }
          }
          // rows j = j0 + g (c0, c1) and j0 + g + 8 (c2, c3); columns i = 8 nt + 2t, +1
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            const int j = j0 + g + 8 * hh;
            float mx = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < BP / 8; ++nt)
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const int i = 8 * nt + 2 * t + e;
                const bool valid = EXACT || (i < b && k * b + i < n_valid);
                const float z = valid ? s[nt][2 * hh + e] * fl : -INFINITY;
                s[nt][2 * hh + e] = z;
                mx = fmaxf(mx, z);
              }
            mx = quad_max(mx);
            float sum = 0.f, sz = 0.f;
#pragma unroll
            for (int nt = 0; nt < BP / 8; ++nt)
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const float z = s[nt][2 * hh + e];
                const float p = ex2(z - mx);                 // 0 for masked columns
                s[nt][2 * hh + e] = p;
                sum += p;
                if (z > -INFINITY) sz = fmaf(p, z, sz);      // 0 log 0 = 0
              }
            sum = quad_sum(sum);
            sz = quad_sum(sz);
            inv_s[rt][hh] = 1.f / sum;
            // c_L = sum R log R (natural log): ln2 * (sum p z / sum - max - log2 sum)
            if (t == 0 && j < b) sCL[k * b + j] = kLn2 * (sz * inv_s[rt][hh] - mx - lg2(sum));
          }
#pragma unroll
          for (int kk = 0; kk < BP / 16; ++kk) {
            pa[rt][kk][0] = Mma<T>::pack(s[2 * kk][0], s[2 * kk][1]);
            pa[rt][kk][1] = Mma<T>::pack(s[2 * kk][2], s[2 * kk][3]);
            pa[rt][kk][2] = Mma<T>::pack(s[2 * kk + 1][0], s[2 * kk + 1][1]);
            pa[rt][kk][3] = Mma<T>::pack(s[2 * kk + 1][2], s[2 * kk + 1][3]);
            if (HILO) {                // what the f16 rounding of the weights left out
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const float2 hi = Mma<T>::unpack(pa[rt][kk][q]);
                const int nt = 2 * kk + (q >> 1), e0 = 2 * (q & 1);
                pal[rt][kk][q] = Mma<T>::pack(s[nt][e0] - hi.x, s[nt][e0 + 1] - hi.y);
              }
            }
          }
        }
        // phase 2: second products, one 16-column slab of v at a time for all row tiles.  This warp
        // alone reads block k of K and V, and every score is formed: on the last round the slab of
        // alpha_L / y goes straight over the slab of K / V it was computed from.
        const uint32_t dstL_u = last ? sK_u : (HILO ? sS_u : sV_u);     // alpha_L of earlier rounds shares V's buffer
        uint32_t v_off[BP / 16];    // rows (k, i) of K and V as the second product's B operand
#pragma unroll
        for (int kk = 0; kk < BP / 16; ++kk) v_off[kk] = rowx<KS>(k, min(16 * kk + (lane & 15), b - 1), b, lane >> 4);
#pragma unroll
        for (int np = 0; np < ksteps; ++np) {   // two 8-column tiles of v per transposing ldmatrix
          uint32_t bk[BP / 16][4], bv[BP / 16][4];
#pragma unroll
          for (int kk = 0; kk < BP / 16; ++kk) {
            ldsm_x4_trans(bk[kk], stp<KS>(sK_u + v_off[kk], np));
            if (last) ldsm_x4_trans(bv[kk], stp<KS>(sV_u + v_off[kk], np));
          }
          __syncwarp();
#pragma unroll
          for (int rt = 0; rt < BP / 16; ++rt) {
            if (16 * rt >= b) continue;
            float o[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            float y[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
            for (int kk = 0; kk < BP / 16; ++kk) {
              Mma<T>::run(o[0], pa[rt][kk], bk[kk]);
              Mma<T>::run(o[1], pa[rt][kk], bk[kk] + 2);
              if (HILO) {
                Mma<T>::run(o[0], pal[rt][kk], bk[kk]);
                Mma<T>::run(o[1], pal[rt][kk], bk[kk] + 2);
              }
              if (last) {
                Mma<T>::run(y[0], pa[rt][kk], bv[kk]);
                Mma<T>::run(y[1], pa[rt][kk], bv[kk] + 2);
              }
            }
            const int j = 16 * rt + st_row;
            const uint32_t off = stp<KS>(rowx<KS>(k, j, b, st_nt), np);
            const float i0 = inv_s[rt][0], i1 = inv_s[rt][1];
            uint32_t hi[4], lo[4];
            split_hilo<HILO>(o[0][0] * i0, o[0][1] * i0, hi[0], lo[0]);
            split_hilo<HILO>(o[0][2] * i1, o[0][3] * i1, hi[1], lo[1]);
            split_hilo<HILO>(o[1][0] * i0, o[1][1] * i0, hi[2], lo[2]);
            split_hilo<HILO>(o[1][2] * i1, o[1][3] * i1, hi[3], lo[3]);
            stsm_x4(j < b ? dstL_u + off : dump_u, hi[0], hi[1], hi[2], hi[3]);
            if (HILO) stsm_x4(j < b ? sALlo_u + off : dump_u, lo[0], lo[1], lo[2], lo[3]);
            if (last)
              stsm_x4(j < b ? sV_u + off : dump_u, Mma<T>::pack(y[0][0] * i0, y[0][1] * i0),
                      Mma<T>::pack(y[0][2] * i1, y[0][3] * i1), Mma<T>::pack(y[1][0] * i0, y[1][1] * i0),
                      Mma<T>::pack(y[1][2] * i1, y[1][3] * i1));
          }
        }
      }
    }
    __syncthreads();

    // ================================================================ L half-step (Eq. 8, 9 / Eq. 4)
    // tile j: Z_L[l,k] = fl * <Q(l,j), alpha_L(k,j)> - c_L(k,j), softmax over k
    {
      const uint32_t sAL_u = last ? sK_u : (HILO ? sS_u : sV_u);      // alpha_L of earlier rounds shares V's buffer
      const uint32_t sAR_u = HILO ? sS_u : sV_u + tile;
      for (int j = warp; j < b; j += nw) {
        float c[MP / 8][2];
#pragma unroll
        for (int nt = 0; nt < MP / 8; ++nt)
#pragma unroll
          for (int e = 0; e < 2; ++e)
            c[nt][e] = sCL[min(8 * nt + 2 * t + e, m - 1) * b + j] * kLog2e;
        float pn[MP / 16][2][MP / 8][2];           // normalised weights [row tile][half][nt][e]
#pragma unroll
        for (int rt = 0; rt < MP / 16; ++rt) {
          const int l0 = 16 * rt;
          if (l0 >= m) {
#pragma unroll
            for (int hh = 0; hh < 2; ++hh)
#pragma unroll
              for (int nt = 0; nt < MP / 8; ++nt) pn[rt][hh][nt][0] = pn[rt][hh][nt][1] = 0.f;
            continue;
          }
          float s[MP / 8][4];
#pragma unroll
          for (int nt = 0; nt < MP / 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) s[nt][e] = 0.f;
          const uint32_t a_u =
              sQ_u + rowx<KS>(min(l0 + (lane & 7) + ((lane >> 3) & 1) * 8, m - 1), j, b, lane >> 4);
          uint32_t b_u[MP / 16];
#pragma unroll
          for (int cp = 0; cp < MP / 16; ++cp)
            b_u[cp] = sAL_u + rowx<KS>(min(16 * cp + (lane & 7) + (lane >> 4) * 8, m - 1), j, b, (lane >> 3) & 1);
#pragma unroll
          for (int ks = 0; ks < ksteps; ++ks) {
            uint32_t a[4];
            ldsm_x4(a, stp<KS>(a_u, ks));
#pragma unroll
            for (int cp = 0; cp < MP / 16; ++cp) {
              uint32_t bf[4];
              ldsm_x4(bf, stp<KS>(b_u[cp], ks));
              Mma<T>::run(s[2 * cp], a, bf);
              Mma<T>::run(s[2 * cp + 1], a, bf + 2);
              if (HILO) {      // + <Q, alpha_L lo>
                ldsm_x4(bf, stp<KS>(b_u[cp] - sAL_u + sALlo_u, ks));
                Mma<T>::run(s[2 * cp], a, bf);
                Mma<T>::run(s[2 * cp + 1], a, bf + 2);
              }
            }
          }
          float inv_s[2];
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            float mx = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < MP / 8; ++nt)
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const float z = (8 * nt + 2 * t + e < m) ? fmaf(s[nt][2 * hh + e], fl, -c[nt][e])
                                                         : -INFINITY;
                s[nt][2 * hh + e] = z;
                mx = fmaxf(mx, z);
              }
            mx = quad_max(mx);
            float sum = 0.f;
#pragma unroll
            for (int nt = 0; nt < MP / 8; ++nt)
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const float p = ex2(s[nt][2 * hh + e] - mx);
                s[nt][2 * hh + e] = p;
                sum += p;
              }
            sum = quad_sum(sum);
            inv_s[hh] = 1.f / sum;
            // log-sum-exp of row b l + j of the final L half-step: summed over a head's rows it is
            // the objective (Eq. 6) at the returned matrix
            if (last && lse != nullptr && t == 0 && l0 + g + 8 * hh < m)
              lse[(size_t)h_idx * N + (size_t)(l0 + g + 8 * hh) * b + j] = (mx + log2f(sum)) * kLn2;
          }
          if (last) {
            // Y(l,j) = sum_k L[j,k,l] y(k,j)   (A = weights rows l, B = y rows (k,j) transposed)
            uint32_t pa[MP / 16][4];
#pragma unroll
            for (int kk = 0; kk < MP / 16; ++kk) {
              pa[kk][0] = Mma<T>::pack(s[2 * kk][0], s[2 * kk][1]);
              pa[kk][1] = Mma<T>::pack(s[2 * kk][2], s[2 * kk][3]);
              pa[kk][2] = Mma<T>::pack(s[2 * kk + 1][0], s[2 * kk + 1][1]);
              pa[kk][3] = Mma<T>::pack(s[2 * kk + 1][2], s[2 * kk + 1][3]);
            }
            uint32_t y_u[MP / 16];
#pragma unroll
            for (int kk = 0; kk < MP / 16; ++kk)
              y_u[kk] = sV_u + rowx<KS>(min(16 * kk + (lane & 15), m - 1), j, b, lane >> 4);
            // only this warp reads the rows (l, j) of Q, and for this row tile it has (they were the
            // A operand of the scores): Y takes their place, slab by slab
            const int l = l0 + st_row;
            const uint32_t row_u = sQ_u + rowx<KS>(l, j, b, st_nt);
            __syncwarp();
#pragma unroll
            for (int np = 0; np < ksteps; ++np) {
              float o[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
              for (int kk = 0; kk < MP / 16; ++kk) {
                uint32_t bf[4];
                ldsm_x4_trans(bf, stp<KS>(y_u[kk], np));
                Mma<T>::run(o[0], pa[kk], bf);
                Mma<T>::run(o[1], pa[kk], bf + 2);
              }
              stsm_x4(l < m ? stp<KS>(row_u, np) : dump_u, Mma<T>::pack(o[0][0] * inv_s[0], o[0][1] * inv_s[0]),
                      Mma<T>::pack(o[0][2] * inv_s[1], o[0][3] * inv_s[1]),
                      Mma<T>::pack(o[1][0] * inv_s[0], o[1][1] * inv_s[0]),
                      Mma<T>::pack(o[1][2] * inv_s[1], o[1][3] * inv_s[1]));
            }
            __syncwarp();
          } else {
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
              const bool row_ok = l0 + g + 8 * hh < m;     // rows past the block must not count
#pragma unroll
              for (int nt = 0; nt < MP / 8; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e)
                  pn[rt][hh][nt][e] = row_ok ? s[nt][2 * hh + e] * inv_s[hh] : 0.f;
            }
          }
        }
        if (last) {
          // the m rows (l, j) of Y are complete: this warp copies them out, 16 bytes per lane
          // (rows of blocks that are absent from a shorter sequence's problem: zeros)
          const int ch = lane & (LPR - 1);
          for (int l = lane / LPR; l < m_alloc; l += RPI) {
            if (ch * 8 >= d) continue;
            const uint4 v = l < m ? *reinterpret_cast<const uint4*>(sQ + at<KS>(l, j, b, ch * 8))
                                  : make_uint4(0u, 0u, 0u, 0u);
            TIn* gp = Y + head_base + (size_t)(l * b + j) * row_stride + ch * 8;
            *reinterpret_cast<uint4*>(gp) = warpmma::from_f16x8(v, gp);
          }
        }
        if (!last) {
          // alpha_R(k,j) = sum_l L[j,k,l] Q(l,j) / c_R, c_R(k,j) = sum_l L[j,k,l]: the contraction
          // runs over the ROW index of the weights, so the A fragments are their transpose.
          // The result does not change when column k is multiplied by any g_k > 0: g_k = 2^-(exponent
          // of the column's largest weight) keeps every column's significant weights in the normal
          // f16 range however small c_R is.
          uint32_t tp[MP / 16][2][MP / 8], tpl[HILO ? MP / 16 : 1][2][HILO ? MP / 8 : 1];
          float cs[MP / 8][2];
#pragma unroll
          for (int nt = 0; nt < MP / 8; ++nt) {
            float gk[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              float cm = 0.f;
#pragma unroll
              for (int rt = 0; rt < MP / 16; ++rt) cm = fmaxf(cm, fmaxf(pn[rt][0][nt][e], pn[rt][1][nt][e]));
              cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 4));
              cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 8));
              cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 16));
              gk[e] = cm > 0.f ? __uint_as_float((253u << 23) - (__float_as_uint(cm) & 0x7f800000u)) : 0.f;
            }
            // column sums of the weights AS ROUNDED to 16 bit: numerator (the MMA below) and
            // denominator of the weighted mean must see the same weights
            float c0 = 0.f, c1 = 0.f;
#pragma unroll
            for (int rt = 0; rt < MP / 16; ++rt)
#pragma unroll
              for (int hh = 0; hh < 2; ++hh) {
                const uint32_t u = Mma<T>::pack(pn[rt][hh][nt][0] * gk[0], pn[rt][hh][nt][1] * gk[1]);
                tp[rt][hh][nt] = u;
                float2 f = Mma<T>::unpack(u);
                if (HILO) {      // the pair carries the weight to 22 bits; c_R sums what the MMAs will see
                  const uint32_t ul = Mma<T>::pack(pn[rt][hh][nt][0] * gk[0] - f.x, pn[rt][hh][nt][1] * gk[1] - f.y);
                  tpl[rt][hh][nt] = ul;
                  const float2 fl2 = Mma<T>::unpack(ul);
                  f.x += fl2.x;
                  f.y += fl2.y;
                }
                c0 += f.x;
                c1 += f.y;
              }
            cs[nt][0] = col_sum(c0);
            cs[nt][1] = col_sum(c1);
          }
#pragma unroll
          for (int kt = 0; kt < MP / 16; ++kt) {
            if (16 * kt >= m) continue;
            // 1 / c_R of rows k = 16 kt + g and + 8: column k = 8 nt + 2 t' + e sits in lane t'
            float ic[2];
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
              const float v0 = __shfl_sync(0xffffffffu, cs[2 * kt + hh][0], g >> 1);
              const float v1 = __shfl_sync(0xffffffffu, cs[2 * kt + hh][1], g >> 1);
              const float cr = (g & 1) ? v1 : v0;
              ic[hh] = cr > 1e-30f ? 1.f / cr : 0.f;
            }
            uint32_t pa[MP / 16][4], pal[HILO ? MP / 16 : 1][4];
#pragma unroll
            for (int ls = 0; ls < MP / 16; ++ls) {
              pa[ls][0] = movm_trans(tp[ls][0][2 * kt]);       // rows k 0-7,  cols l 0-7
              pa[ls][1] = movm_trans(tp[ls][0][2 * kt + 1]);   // rows k 8-15, cols l 0-7
              pa[ls][2] = movm_trans(tp[ls][1][2 * kt]);       // rows k 0-7,  cols l 8-15
              pa[ls][3] = movm_trans(tp[ls][1][2 * kt + 1]);   // rows k 8-15, cols l 8-15
              if (HILO) {
                pal[ls][0] = movm_trans(tpl[ls][0][2 * kt]);
                pal[ls][1] = movm_trans(tpl[ls][0][2 * kt + 1]);
                pal[ls][2] = movm_trans(tpl[ls][1][2 * kt]);
                pal[ls][3] = movm_trans(tpl[ls][1][2 * kt + 1]);
              }
            }
            uint32_t q_u[MP / 16];
#pragma unroll
            for (int ls = 0; ls < MP / 16; ++ls)
              q_u[ls] = sQ_u + rowx<KS>(min(16 * ls + (lane & 15), m - 1), j, b, lane >> 4);
            const int kr = 16 * kt + st_row;                   // alpha_R row (kr, j) this lane addresses
            const uint32_t row_u = sAR_u + rowx<KS>(kr, j, b, st_nt);
#pragma unroll
            for (int np = 0; np < ksteps; ++np) {
              float o[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
              for (int ls = 0; ls < MP / 16; ++ls) {
                uint32_t bf[4];   // B[kk = l][n = v] = Q(l,j)[v], read transposed; two 8-column tiles
                ldsm_x4_trans(bf, stp<KS>(q_u[ls], np));
                Mma<T>::run(o[0], pa[ls], bf);
                Mma<T>::run(o[1], pa[ls], bf + 2);
                if (HILO) {
                  Mma<T>::run(o[0], pal[ls], bf);
                  Mma<T>::run(o[1], pal[ls], bf + 2);
                }
              }
              uint32_t hi[4], lo[4];
              split_hilo<HILO>(o[0][0] * ic[0], o[0][1] * ic[0], hi[0], lo[0]);
              split_hilo<HILO>(o[0][2] * ic[1], o[0][3] * ic[1], hi[1], lo[1]);
              split_hilo<HILO>(o[1][0] * ic[0], o[1][1] * ic[0], hi[2], lo[2]);
              split_hilo<HILO>(o[1][2] * ic[1], o[1][3] * ic[1], hi[3], lo[3]);
              stsm_x4(kr < m ? stp<KS>(row_u, np) : dump_u, hi[0], hi[1], hi[2], hi[3]);
              if (HILO) stsm_x4(kr < m ? stp<KS>(row_u - sAR_u + sARlo_u, np) : dump_u, lo[0], lo[1], lo[2], lo[3]);
            }
          }
        }
      }
    }
    __syncthreads();
  }

}

inline bool supported(int N, int d, int b, int m, int dtype, int T) {
  return (dtype == 1 || dtype == 2) && d % 8 == 0 && d <= 128 && b <= (d <= 64 ? 64 : 32) && m <= 32 &&
         smem_bytes(N, T, kThreads, b, ksteps_for(d)) <= (size_t)kMaxSmem;
}

// Three or more rounds with hi + lo states: blocks and block counts up to 16, d <= 80, five tiles in
// shared memory.
inline bool supported_hilo(int N, int d, int b, int m, int dtype, int T) {
  return (dtype == 1 || dtype == 2) && T >= 3 && d % 8 == 0 && d <= 80 && b <= 16 && m <= 16 &&
         smem_bytes(N, T, kThreads, b, ksteps_for(d), true) <= (size_t)kMaxSmem;
}

int launch(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int d, int b,
           int m, int T, int dtype, float scale, int n_valid, int H, float* lse, cudaStream_t st,
           const int* seq_len = nullptr, int heads = 1);

#ifdef MA_TU_FUSED_SMALL
template <typename TIn, int BP, int MP, bool EXACT = false, int KS = 4, bool HILO = false>
inline int launch_t(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int d, int b,
                    int m, int T, float scale, int n_valid, int H, float* lse, cudaStream_t st,
                    const int* seq_len, int heads) {
  auto kern = monarch_fused_small<TIn, BP, MP, EXACT, KS, HILO>;
  // The 16 x 16 kernel is compiled for 128 registers: two CTAs of 8 warps per SM where shared memory
  // lets two fit, else one CTA of 16 warps (each warp then owns at most one tile per half-step).
  int threads = kThreads;
  if (KS == 4 && !HILO && BP <= 32 && (BP == 16 || MP == 16) && 2 * (smem_bytes(N, T) + 1024) > (size_t)228 * 1024 &&
      (m > 8 || b > 8) && smem_bytes(N, T, 2 * kThreads) <= (size_t)kMaxSmem)
    threads = 2 * kThreads;
  const size_t smem = smem_bytes(N, T, threads, b, KS, HILO);
  if (cudaFuncSetAttribute((const void*)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
      cudaSuccess)
    return 7;
  // programmatic stream serialisation: when calls follow one another on a stream, the CTAs of the
  // next call take SM slots while the last wave of this one drains (they touch no memory before
  // this launch has finished: the kernel starts with griddepcontrol.wait)
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(BH);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, (const TIn*)Q, (const TIn*)K, (const TIn*)V, (TIn*)Y, N, d, b, m, T, scale,
                            n_valid, H, lse, seq_len, heads) == cudaSuccess
             ? 0
             : 7;
}

template <typename TIn>
inline int launch_d(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int d, int b,
                    int m, int T, float scale, int n_valid, int H, float* lse, cudaStream_t st,
                    const int* seq_len, int heads) {
#define MA_FS_ARGS Q, K, V, Y, BH, N, d, b, m, T, scale, n_valid, H, lse, st, seq_len, heads
  if (supported_hilo(N, d, b, m, 1, T))   // three or more rounds: hi + lo states
    return d <= 64 ? launch_t<TIn, 16, 16, false, 4, true>(MA_FS_ARGS) : launch_t<TIn, 16, 16, false, 5, true>(MA_FS_ARGS);
  if (d == 64 && n_valid >= N && seq_len == nullptr) {   // exact fits, no mask
    if (b == 16 && m == 16) return launch_t<TIn, 16, 16, true>(MA_FS_ARGS);
    if (b == 32 && m == 32) return launch_t<TIn, 32, 32, true>(MA_FS_ARGS);
    if (b == 16 && m == 32) return launch_t<TIn, 16, 32, true>(MA_FS_ARGS);
    if (b == 32 && m == 16) return launch_t<TIn, 32, 16, true>(MA_FS_ARGS);
  }
  if (d > 80) {          // rows of up to 128 columns
    if (b <= 16) return m <= 16 ? launch_t<TIn, 16, 16, false, 8>(MA_FS_ARGS) : launch_t<TIn, 16, 32, false, 8>(MA_FS_ARGS);
    return m <= 16 ? launch_t<TIn, 32, 16, false, 8>(MA_FS_ARGS) : launch_t<TIn, 32, 32, false, 8>(MA_FS_ARGS);
  }
  if (d > 64) {          // rows of up to 80 columns (d = 72)
    if (b <= 16) return m <= 16 ? launch_t<TIn, 16, 16, false, 5>(MA_FS_ARGS) : launch_t<TIn, 16, 32, false, 5>(MA_FS_ARGS);
    return m <= 16 ? launch_t<TIn, 32, 16, false, 5>(MA_FS_ARGS) : launch_t<TIn, 32, 32, false, 5>(MA_FS_ARGS);
  }
  if (b > 48) return m <= 16 ? launch_t<TIn, 64, 16>(MA_FS_ARGS) : launch_t<TIn, 64, 32>(MA_FS_ARGS);
  if (b > 32) return m <= 16 ? launch_t<TIn, 48, 16>(MA_FS_ARGS) : launch_t<TIn, 48, 32>(MA_FS_ARGS);
  if (b <= 16 && m <= 16) return launch_t<TIn, 16, 16>(MA_FS_ARGS);
  if (b <= 16) return launch_t<TIn, 16, 32>(MA_FS_ARGS);
  if (m <= 16) return launch_t<TIn, 32, 16>(MA_FS_ARGS);
  return launch_t<TIn, 32, 32>(MA_FS_ARGS);
#undef MA_FS_ARGS
}

int launch(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int d, int b,
           int m, int T, int dtype, float scale, int n_valid, int H, float* lse, cudaStream_t st,
           const int* seq_len, int heads) {
  if (dtype == 1)
    return launch_d<__half>(Q, K, V, Y, BH, N, d, b, m, T, scale, n_valid, H, lse, st, seq_len, heads);
  return launch_d<__nv_bfloat16>(Q, K, V, Y, BH, N, d, b, m, T, scale, n_valid, H, lse, st, seq_len, heads);
}

#endif  // MA_TU_FUSED_SMALL

}  // namespace fsmall
}  // namespace ma
