// Translation unit of fused_small.cuh: defines what that header only declares elsewhere.
#define MA_TU_FUSED_SMALL
#include "fused_small.cuh"
