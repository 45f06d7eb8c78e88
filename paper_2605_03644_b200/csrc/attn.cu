// placeholder until the tcgen05 kernel lands
#include "common.cuh"
extern "C" size_t adapshot_attn_workspace_bytes(const adapshot_model_t*, int32_t, int32_t, int32_t, int32_t, int64_t) { return 0; }
extern "C" int adapshot_query_attn(const adapshot_model_t*, const void*, const void*, int64_t, const int64_t*, int32_t, int32_t,
                                   const int32_t*, int32_t, const void*, const void*, const void*, int32_t, int32_t, int32_t,
                                   void*, float*, uint32_t, void*, size_t, int32_t*, void*) { return ADAPSHOT_EUNSUPPORTED; }
