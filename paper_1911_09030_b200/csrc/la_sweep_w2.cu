// Two replicas: four coordinates per thread (see la_sweep_w1.cu), both replicas in one chunk.
#define LA_W 2
#define LA_VEC 4
#define LA_CH_V4 2
#define LA_PERIOD_VEC 2
#include "la_sweep_inst.inc"
