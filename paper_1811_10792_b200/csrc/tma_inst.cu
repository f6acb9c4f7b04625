// Pipelined (bulk-copy) step kernels, fused diagnostics off.
#define SGP_INST_DIAG false
#include "tma_instances.inc"
