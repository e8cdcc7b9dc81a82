#define LA_W 1
#include "la_sweep_inst.inc"
