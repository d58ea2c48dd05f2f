// slim_mpq_gemm: batched path (M > 16).  Placeholder until the tcgen05 kernel lands.
#include "slim_common.cuh"

extern "C" int slim_mpq_gemm(const void*, const void*, const uint8_t*, const void*, const void*, void*,
                             int, int, int, int, void*, size_t, void*) {
    return SLIM_ERR_UNSUPPORTED;
}
