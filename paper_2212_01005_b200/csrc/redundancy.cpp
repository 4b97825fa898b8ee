// Host-side redundancy calculator for intensive fusion (Section III-B): upstream work with and
// without fusion for a given downstream tiling, in closed form per dimension.
#include <cstdint>
#include <string>

#include "../../include/ago.h"

namespace ago {
ago_status_t report_failure(ago_status_t s, const char* msg);   // records the thread's last error (api.cu)
}

namespace {

// Sum over the tiles of one downstream dimension (extent D, tile d) of the upstream extent each
// tile needs: a tile of t outputs with window K and stride s reads (t - 1) * s + K inputs.
int64_t needed_extent_sum(int64_t D, int64_t d, int64_t K, int64_t s, int64_t* tiles) {
  if (d > D) d = D;
  const int64_t full = D / d, tail = D - full * d;
  *tiles = full + (tail ? 1 : 0);
  int64_t sum = full * ((d - 1) * s + K);
  if (tail) sum += (tail - 1) * s + K;
  return sum;
}

}  // namespace

extern "C" ago_status_t ago_fusion_redundancy(const ago_redundancy_query_t* q, ago_redundancy_result_t* out) {
  auto fail = [](ago_status_t st, const char* msg) { return ago::report_failure(st, msg); };
  if (!q || !out) return fail(AGO_ERR_INVALID_ARG, "ago_fusion_redundancy: NULL argument");
  if (q->struct_size != sizeof(ago_redundancy_query_t)) return fail(AGO_ERR_INVALID_ARG, "ago_fusion_redundancy: struct_size mismatch");
  const int64_t v[] = {q->N, q->O1, q->I1, q->R1, q->C1, q->O2, q->R2, q->C2, q->stride2, q->H2, q->W2, q->o2, q->h2, q->w2};
  for (int64_t x : v)
    if (x <= 0) return fail(AGO_ERR_INVALID_ARG, "ago_fusion_redundancy: every extent must be positive");
  if (q->depthwise2 && q->O2 != q->O1) return fail(AGO_ERR_SHAPE, "ago_fusion_redundancy: a depthwise downstream operator needs O2 == O1");

  const int64_t H1 = (q->H2 - 1) * q->stride2 + q->R2, W1 = (q->W2 - 1) * q->stride2 + q->C2;
  int64_t th = 0, tw = 0, tc = 0;
  const int64_t hsum = needed_extent_sum(q->H2, q->h2, q->R2, q->stride2, &th);
  const int64_t wsum = needed_extent_sum(q->W2, q->w2, q->C2, q->stride2, &tw);
  // channels: a dense downstream tile needs all O1 upstream channels; a depthwise tile its own
  const int64_t o2 = q->o2 > q->O2 ? q->O2 : q->o2;
  tc = (q->O2 + o2 - 1) / o2;
  const int64_t csum = q->depthwise2 ? q->O1 : tc * q->O1;

  out->num_tiles = q->N * tc * th * tw;
  out->upstream_elems_unfused = q->N * q->O1 * H1 * W1;
  out->upstream_elems_fused = q->N * csum * hsum * wsum;
  const int64_t red = q->I1 * q->R1 * q->C1;
  out->upstream_macs_unfused = out->upstream_elems_unfused * red;
  out->upstream_macs_fused = out->upstream_elems_fused * red;
  out->factor = (double)out->upstream_elems_fused / (double)out->upstream_elems_unfused;
  out->category = q->depthwise2 ? AGO_LINK_DOWNSTREAM_DEPTHWISE
                                : ((q->R2 == 1 && q->C2 == 1 && q->stride2 == 1) ? AGO_LINK_DOWNSTREAM_POINTWISE : AGO_LINK_GENERAL);
  out->reserved = 0;
  return AGO_OK;
}
