// Placeholder until the tensor-core kernels are linked in: reports every shape as unsupported.
#include "common.cuh"
int fs_tc_supported(const fsharp_dims*, int, int, int, float) { return 0; }
size_t fs_tc_attend_scratch_bytes(const fsharp_ctx*, const fsharp_dims*, int, int) { return 0; }
int fs_tc_attend(fsharp_ctx*, const void*, const void*, const void*, const fsharp_dims*, int, int, const float*, void*,
                 WsAlloc*) { return FSHARP_E_SHAPE; }
