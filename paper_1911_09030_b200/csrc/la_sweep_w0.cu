#define LA_W 0
#include "la_sweep_inst.inc"
