// Worker count known only at run time: the counter-form reduction tree keeps one partial sum per
// level in registers, so these kernels get the larger register budget (two blocks per SM).
#define LA_W 0
#define LA_MINB 2
#include "la_sweep_inst.inc"
