// Translation unit of fused_f32.cuh: defines what that header only declares elsewhere.
#define MA_TU_FUSED_F32
#include "fused_f32.cuh"
