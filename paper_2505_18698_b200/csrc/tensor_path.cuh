// Tensor-core (tcgen05 + TMA) path: interface used by the C-ABI layer.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

namespace ma {
namespace tensor {

inline bool supported(int N, int d, int b, int m, int dtype, int BH) { return false; }
inline size_t workspace_bytes(int BH, int N, int d, int b, int T) { return 0; }
inline int launch(const void* Q, const void* K, const void* V, void* Y, int BH, int N, int d, int b,
                  int T, int dtype, float scale, void* ws, cudaStream_t st, int* launches) {
  return 4;  // MA_ERR_UNSUPPORTED
}

}  // namespace tensor
}  // namespace ma
