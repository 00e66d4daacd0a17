// Host-side schedule helpers of SFB (no device code): the Halton-sequence partial broadcast of
// Section 4.3 and the stale-synchronous rule of Section 4.1.  They decide which worker streams a
// worker would send and when it may start its next batch; nothing here touches the GPU.
#include "sfb.h"

extern "C" int sfb_halton_peers(int32_t P, int32_t Q, int32_t p, int32_t* peers) {
  if (peers == nullptr || P <= 0 || Q < 0 || p < 0 || p >= P) return SFB_ERR_ARG;
  // offsets floor(P * f) for f = 1/2, 1/4, 3/4, 1/8, 3/8, 5/8, 7/8, ...
  int n = 0;
  for (long long den = 2; n < Q; den *= 2) {
    if (den > (1ll << 40)) return SFB_ERR_SHAPE;
    for (long long num = 1; num < den && n < Q; num += 2) {
      const long long off = (num * (long long)P) / den;
      peers[n++] = (int32_t)(((long long)p + off) % P);
    }
  }
  return SFB_OK;
}

extern "C" int sfb_ssp_may_proceed(int64_t t_p, const int64_t* tau, int32_t P, int64_t staleness) {
  if (tau == nullptr || P <= 0) return SFB_ERR_ARG;
  if (staleness < 0) return 1;   // negative = unbounded staleness (ASP)
  for (int32_t q = 0; q < P; ++q)
    if (t_p - tau[q] > staleness) return 0;
  return 1;
}
