// Six replicas as ONE chunk.  Pure-noise gradients fit 80 registers and keep three blocks resident
// (K1 0.93 -> 1.01, K3 0.91 -> 1.00 of the copy bandwidth); the problem arrays of the scaled noise and of the
// quadratic and an fp32 table's chunk of rows spill at that budget and keep two blocks (quadratic K1
// 5.85 against 6.39 TB/s, scaled noise 6.18 against 6.43).
#define LA_W 6
#define LA_CH 6
#define LA_MINB 3
#define LA_MINB_SCALED 2
#define LA_MINB_QUADRATIC 2
#define LA_MINB_TABLE 2
#define LA_PERIOD_MINB 3
#include "la_sweep_inst.inc"
