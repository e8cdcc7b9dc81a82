#define LA_W 3
#include "la_sweep_inst.inc"
