#define LA_W 4
// The step that reads the one stored copy of the sums and writes every replica is write-heavy:
// 128-bit stores measured 4 to 7 % faster there; every other pass keeps two coordinates per thread.
#define LA_IMPORT_VEC 4
// bf16 gradient table (four coordinates per thread): with only four replicas the averaging passes
// take them two per chunk (K3 0.98, sums-only step 0.96 of the copy bandwidth against 0.95, 0.92 with one).
#define LA_CH_V4 2
#include "la_sweep_inst.inc"
