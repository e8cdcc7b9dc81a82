#define LA_W 9
#include "la_sweep_inst.inc"
