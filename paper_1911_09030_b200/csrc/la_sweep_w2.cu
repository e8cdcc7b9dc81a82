#define LA_W 2
#include "la_sweep_inst.inc"
