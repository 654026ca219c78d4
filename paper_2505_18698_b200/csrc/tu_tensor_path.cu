// Translation unit of tensor_path.cuh: defines what that header only declares elsewhere.
#define MA_TU_TENSOR_BASIC
#include "tensor_path.cuh"
