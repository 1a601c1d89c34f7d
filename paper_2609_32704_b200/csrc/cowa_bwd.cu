// CoWindow Attention backward (Algorithm 2) -- placeholder until the kernels land.
#include "cowa_common.h"

extern "C" {

size_t cowa_bwd_workspace_bytes(int B, int T, int Hq, int Hkv, int D, const cowa_params_t* p) {
  (void)Hkv; (void)D; (void)p;
  if (B <= 0 || T <= 0 || Hq <= 0) return 0;
  return (size_t)B * Hq * T * sizeof(float);
}

int cowa_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
             void* dq, void* dk, void* dv, int B, int T, int Hq, int Hkv, int D, const cowa_params_t* p,
             void* workspace, size_t workspace_bytes, void* stream) {
  (void)T; (void)B; (void)Hq; (void)Hkv; (void)D; (void)workspace_bytes; (void)stream;
  if (!q || !k || !v || !o || !lse || !d_o || !dq || !dk || !dv || !p || !workspace) return COWA_ERR_INVALID_ARG;
  return COWA_ERR_UNSUPPORTED;
}

}  // extern "C"
