#include "tc.h"

namespace dc {

struct TcState { const char* err = ""; };

bool tc_supported(const dc_config&) { return false; }
int tc_create(const dc_config&, cudaStream_t, int, int, const std::vector<const void*>&,
              const std::vector<const void*>&, const std::vector<const void*>&,
              const std::vector<const void*>&, const std::vector<const void*>&,
              const std::vector<const void*>&, const std::vector<const void*>&, const void*,
              TcState** out) { *out = nullptr; return DC_ERR_UNSUPPORTED; }
void tc_destroy(TcState* t) { delete t; }
const char* tc_error(const TcState* t) { return t ? t->err : ""; }
int tc_layer(TcState*, int, const SeqMeta&, float*, const __nv_bfloat16*, const __nv_bfloat16*,
             const __nv_bfloat16*, const float*, const __nv_bfloat16*, const float**, int*,
             size_t*, StageHook&) { return DC_ERR_UNSUPPORTED; }
int tc_lmhead(TcState*, const SeqMeta&, const __nv_bfloat16*, int, int, int32_t*, float*, float*,
              float*, float*, SignalOut) { return DC_ERR_UNSUPPORTED; }

}  // namespace dc
