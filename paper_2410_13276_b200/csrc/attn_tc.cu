// placeholder until the tcgen05 kernel lands: reports failure so nothing silently runs another path
#include "seer_internal.cuh"
namespace seer {
seer_status init_attn_tc(seer_ctx*) { return SEER_OK; }
int launch_attn_tc(seer_ctx*, const SeqMeta&, const void*, const void*, const void*, const int32_t*, const int32_t*, void*,
                   float*, cudaStream_t) { return -(int)cudaErrorNotSupported; }
}  // namespace seer
