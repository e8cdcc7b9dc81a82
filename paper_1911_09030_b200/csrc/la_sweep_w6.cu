#define LA_W 6
#include "la_sweep_inst.inc"
