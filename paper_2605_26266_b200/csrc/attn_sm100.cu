// Corrected chunk attention, tcgen05/TMEM kernel for sm_100a (placeholder until the kernel lands).
#include "kvq_common.cuh"

namespace kvq {

bool attn_tcgen05_supports(const kvq_cache_desc*, int64_t, int64_t) { return false; }
size_t attn_tcgen05_workspace_bytes(const kvq_cache_desc*, int64_t, int64_t, int64_t) { return 0; }
int launch_attn_tcgen05(const AttnArgs&) { return KVQ_ERR_UNSUPPORTED; }

}  // namespace kvq
