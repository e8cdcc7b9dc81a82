#define LA_W 64
#include "la_sweep_inst.inc"
