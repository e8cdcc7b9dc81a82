#define LA_W 7
#include "la_sweep_inst.inc"
