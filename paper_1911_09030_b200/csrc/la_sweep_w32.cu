#define LA_W 32
#include "la_sweep_inst.inc"
