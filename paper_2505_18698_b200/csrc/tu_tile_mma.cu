// Translation unit of tile_mma.cuh: defines what that header only declares elsewhere.
#define MA_TU_TILE_MMA
#include "tile_mma.cuh"
