// Register-staged step kernels, vector width 4, fused diagnostics off.
#define SGP_INST_VEC 4
#define SGP_INST_DIAG false
#include "regs_instances.inc"
