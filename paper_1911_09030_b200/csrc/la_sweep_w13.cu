#define LA_W 13
#include "la_sweep_inst.inc"
