// Five replicas as ONE chunk (a chunk of four would leave a single replica in flight behind it);
// with generated gradients that still fits 80 registers, so three blocks stay resident (with two:
// K1 0.91, K3 0.89 of the copy bandwidth; with three 1.00, 1.00).  An fp32 table's chunk of rows
// does not fit: two blocks there (K1 1.03 against 0.97 with three), and the stand-alone average
// measured 2 % faster at N = 2^26 with two.
#define LA_W 5
#define LA_CH 5
#define LA_MINB 3
#define LA_MINB_TABLE 2
#define LA_MINB_SYNC 2
#define LA_PERIOD_MINB 3
#include "la_sweep_inst.inc"
