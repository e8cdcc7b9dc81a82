// One replica gives a two-coordinate thread only 16 bytes of x and B^2 to fetch per group: four
// coordinates per thread, so that enough loads are in flight to cover the memory latency.
#define LA_W 1
#define LA_VEC 4
#define LA_MINB 4  // 64 registers are enough for one replica: a fourth resident block (K1 0.91 -> 0.99 of the copy bandwidth)
#define LA_BF16_MINB 3
#define LA_PERIOD_MINB 3
#define LA_PERIOD_VEC 2
#include "la_sweep_inst.inc"
