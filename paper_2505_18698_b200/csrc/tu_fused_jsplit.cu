// Translation unit of fused_jsplit.cuh: defines what that header only declares elsewhere.
#define MA_TU_FUSED_JSPLIT
#include "fused_jsplit.cuh"
