#define LA_W 16
#include "la_sweep_inst.inc"
