// Three replicas give a two-coordinate thread only 48 bytes of loads in flight, too few to cover
// the memory latency: four coordinates per thread (and the register budget that needs).
#define LA_W 3
#define LA_VEC 4
#define LA_CH_V4 3
#define LA_MINB 2
#define LA_BF16_MINB 2
#define LA_PERIOD_VEC 2
#define LA_PERIOD_MINB 3
#include "la_sweep_inst.inc"
