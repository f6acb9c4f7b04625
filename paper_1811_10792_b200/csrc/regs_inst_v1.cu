// Register-staged step kernels, vector width 1, fused diagnostics off.
#define SGP_INST_VEC 1
#define SGP_INST_DIAG false
#include "regs_instances.inc"
