// Five replicas as ONE chunk (a chunk of four would leave a single replica in flight behind it).
#define LA_W 5
#define LA_CH 5
#define LA_MINB 2
#define LA_PERIOD_MINB 3
#include "la_sweep_inst.inc"
