// tcgen05 cross-attention kernel (placeholder interface; body follows in this header).
#pragma once
#include "common.cuh"
#include "tc.cuh"

namespace grace {

inline bool cross_attn_tc_supported(int B, int M, int H, int d_h, int T_ctx) {
  (void)B; (void)M; (void)H; (void)d_h; (void)T_ctx;
  return false;
}

inline grace_status_t launch_cross_attn_tc(const uint16_t*, int64_t, const uint16_t*, const uint16_t*, int64_t,
                                           int64_t, int64_t, uint16_t*, int64_t, float*, int, int, int, int, int,
                                           float, cudaStream_t) {
  return GRACE_UNSUPPORTED_SHAPE;
}

}  // namespace grace
