// Six replicas as ONE chunk (chunks of four would leave a half-empty second chunk in flight).
#define LA_W 6
#define LA_CH 6
#define LA_MINB 2
#define LA_PERIOD_MINB 3
#include "la_sweep_inst.inc"
