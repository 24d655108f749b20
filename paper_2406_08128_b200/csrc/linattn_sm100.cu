// placeholder until the tensor-core kernel lands
#include "common.cuh"
namespace chela {
bool linattn_sm100_supported(int, int, int, int, int, chela_dtype_t, chela_dtype_t) { return false; }
size_t linattn_sm100_workspace_bytes(int, int, int, int, int) { return 0; }
chela_status_t launch_linattn_sm100(const void *, const void *, const void *, void *, int, int, int, int, int,
                                    chela_dtype_t, chela_dtype_t, int, float, float, void *, cudaStream_t)
{
    return CHELA_ERR_UNSUPPORTED;
}
}  // namespace chela
