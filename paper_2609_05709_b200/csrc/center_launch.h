// Dispatch of the per-centre kernel over its compile-time l_max (0..12).
#pragma once
#include "soap_device.cuh"

namespace soap {
cudaError_t center_set_smem(bool deriv, int l_max, int bytes);
cudaError_t center_launch(bool deriv, int l_max, const CenterParams& p, unsigned grid, size_t smem, cudaStream_t st);
// one group of l_max values per translation unit, so that they compile in parallel
cudaError_t center_set_smem_g0(bool, int, int);  cudaError_t center_launch_g0(bool, int, const CenterParams&, unsigned, size_t, cudaStream_t);
cudaError_t center_set_smem_g1(bool, int, int);  cudaError_t center_launch_g1(bool, int, const CenterParams&, unsigned, size_t, cudaStream_t);
cudaError_t center_set_smem_g2(bool, int, int);  cudaError_t center_launch_g2(bool, int, const CenterParams&, unsigned, size_t, cudaStream_t);
cudaError_t center_set_smem_g3(bool, int, int);  cudaError_t center_launch_g3(bool, int, const CenterParams&, unsigned, size_t, cudaStream_t);
}  // namespace soap
