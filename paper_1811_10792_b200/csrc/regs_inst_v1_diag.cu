// Register-staged step kernels, vector width 1, fused diagnostics on.
#define SGP_INST_VEC 1
#define SGP_INST_DIAG true
#include "regs_instances.inc"
