// Translation unit of tensor_tmem.cuh: defines what that header only declares elsewhere.
#define MA_TU_TENSOR_TMEM
#include "tensor_tmem.cuh"
