// Placeholder until the tcgen05 kernel lands: reports that no shape is supported, so that
// AMX_GEMM_AUTO picks the SIMT kernel and AMX_GEMM_TC returns AMX_ERR_SHAPE.
#include "gemm.cuh"

namespace amx {

bool gemm_tc_supported(int64_t, int64_t, int64_t, int) { return false; }
size_t gemm_tc_workspace_bytes(int64_t, int64_t, int64_t) { return 0; }
int gemm_tc(const uint8_t*, const uint8_t*, const uint8_t*, const uint8_t*, int64_t, int64_t,
            int64_t, float*, int64_t, void*, cudaStream_t) { return AMX_ERR_SHAPE; }
int gemm_tc_status(const void*, cudaStream_t) { return AMX_OK; }

}  // namespace amx
