/* Plain C99 client of the C ABI: compiles the one-peer exponential schedule for n nodes and prints, for
 * every step of one period, the in-neighbour lists with their weights.  Built and run by the tests to
 * show that include/sgp.h is a valid C header and that the library links from C without a GPU. */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "sgp.h"

int main(int argc, char **argv) {
  int n = argc > 1 ? atoi(argv[1]) : 8;
  sgp_graph_desc g;
  sgp_schedule *s = NULL;
  int64_t period = 0, nnz = 0, k;
  int32_t rowptr[SGP_MAX_NODES + 1], col[4 * SGP_MAX_NODES];
  float val[4 * SGP_MAX_NODES];
  int rc, i, e;

  memset(&g, 0, sizeof g);
  g.kind = SGP_GRAPH_EXP_PEERS;
  g.peers = 1;
  rc = sgp_schedule_compile(&s, n, &g);
  if (rc != SGP_OK) {
    printf("error %d: %s\n", rc, sgp_strerror(rc));
    return 1;
  }
  sgp_schedule_period(s, &period);
  printf("version %d n %d period %lld\n", sgp_version(), n, (long long)period);
  for (k = 0; k < period; ++k) {
    rc = sgp_schedule_get(s, k, rowptr, col, val, 4 * SGP_MAX_NODES, &nnz);
    if (rc != SGP_OK) return 2;
    for (i = 0; i < n; ++i)
      for (e = rowptr[i]; e < rowptr[i + 1]; ++e) printf("%lld %d %d %.9g\n", (long long)k, i, col[e], (double)val[e]);
  }
  sgp_schedule_destroy(s);
  /* error paths */
  g.peers = 0;
  if (sgp_schedule_compile(&s, n, &g) != SGP_ERR_ARG || s != NULL) return 3;
  if (sgp_step(NULL, NULL, NULL, NULL, NULL, NULL, 0, 0.1f, 0.0f, 0.0f, 1, NULL) != SGP_ERR_ARG) return 4;
  return 0;
}
