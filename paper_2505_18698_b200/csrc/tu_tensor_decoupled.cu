// Translation unit of tensor_decoupled.cuh: defines what that header only declares elsewhere.
#define MA_TU_TENSOR_DECOUPLED
#include "tensor_decoupled.cuh"
