// Translation unit of tensor_persistent.cuh: defines what that header only declares elsewhere.
#define MA_TU_TENSOR_PERSISTENT
#include "tensor_persistent.cuh"
