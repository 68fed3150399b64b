// placeholder, replaced by the MLP kernels
#pragma once
#include "linear_kernel.cuh"
namespace ssim {
struct MlpScratch { void* p = nullptr; };
inline const char* mlp_shape_unsupported(int, int, int, int) { return "mlp kernel not built"; }
inline cudaError_t mlp_scratch_alloc(MlpScratch&, int, int, int, int, int, int, int, bool, cudaStream_t) { return cudaSuccess; }
inline void mlp_scratch_free(MlpScratch&) {}
inline cudaError_t mlp_after_set_params(MlpScratch&, float*, long long, int, cudaStream_t) { return cudaSuccess; }
inline cudaError_t run_mlp(NumericArgs&, MlpScratch&, int, int, cudaStream_t, const char** why) { *why = "mlp kernel not built"; return cudaSuccess; }
}
