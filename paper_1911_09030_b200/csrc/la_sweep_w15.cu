#define LA_W 15
#include "la_sweep_inst.inc"
