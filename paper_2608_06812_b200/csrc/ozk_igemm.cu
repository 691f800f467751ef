// INT8 x INT8 -> INT32 on FP4 limbs (Section 3, last paragraph; Eq. 1 with p = q = 3).
#include "ozk_common.cuh"

extern "C" {

size_t ozk_igemm_i8_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  (void)M; (void)N; (void)K;
  return 0;
}

ozk_status ozk_igemm_i8(int64_t, int64_t, int64_t, const int8_t*, int64_t, const int8_t*, int64_t, int32_t*, int64_t, void*) {
  return OZK_ERR_UNSUPPORTED;
}

}  // extern "C"
