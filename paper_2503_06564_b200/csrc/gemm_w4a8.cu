// W4A8 variant of the integer GEMM (int4 weights with one scale per 128 consecutive k).
#include "internal.h"

namespace trdq {

trdq_status launch_gemm_w4(const trdq_weights*, int, const GemmSegment*, const void*, cudaStream_t) {
  return TRDQ_ERR_WBITS;
}

}  // namespace trdq
