// Pipelined (bulk-copy) step kernels, fused diagnostics on.
#define SGP_INST_DIAG true
#include "tma_instances.inc"
