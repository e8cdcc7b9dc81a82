#define LA_W 14
#include "la_sweep_inst.inc"
