#define LA_W 8
#include "la_sweep_inst.inc"
