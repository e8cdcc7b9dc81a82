#define LA_W 10
#include "la_sweep_inst.inc"
