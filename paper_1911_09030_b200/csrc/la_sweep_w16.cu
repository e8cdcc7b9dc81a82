#define LA_W 16
// The step that reads the one stored copy of the sums and writes every replica is write-heavy:
// 128-bit stores measured 4 to 7 % faster there; every other pass keeps two coordinates per thread.
#define LA_IMPORT_VEC 4
#include "la_sweep_inst.inc"
