#define LA_W 11
#include "la_sweep_inst.inc"
