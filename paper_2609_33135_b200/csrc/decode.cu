// placeholder until the decode kernel lands
#include "common.cuh"
using namespace mpfa;
extern "C" size_t mpfa_decode_workspace_bytes(int B, int H_q, int H_kv, int max_pages_per_req) {
  (void)B; (void)H_q; (void)H_kv; (void)max_pages_per_req;
  return 0;
}
extern "C" mpfa_status mpfa_decode(const mpfa_fp4_tensor *, const mpfa_paged_kv *, const int32_t *, int, const int32_t *,
                                   const mpfa_stats *, float, float, void *, float *, void *, size_t, int32_t *, void *) {
  return MPFA_ERR_UNSUPPORTED;
}
