#define LA_W 12
#include "la_sweep_inst.inc"
