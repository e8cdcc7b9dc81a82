#define LA_W 4
#include "la_sweep_inst.inc"
