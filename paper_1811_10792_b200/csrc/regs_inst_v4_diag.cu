// Register-staged step kernels, vector width 4, fused diagnostics on.
#define SGP_INST_VEC 4
#define SGP_INST_DIAG true
#include "regs_instances.inc"
