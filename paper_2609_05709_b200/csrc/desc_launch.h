// Dispatch of the descriptor-only kernel over its compile-time l_max (0..12) and padded n_max (4, 8, 12, 16).
#pragma once
#include "soap_device.cuh"

namespace soap {
// harmonic normalisation up to l = 12: anorm[91] (index l(l+1)/2 + m)
cudaError_t desc_constants(int l_max, const float* anorm91);
cudaError_t desc_set_smem(int l_max, int np, int bytes);
// plain: every option at its default (see desc_kernel); table_in_smem: the radial table is staged per CTA
cudaError_t desc_launch(int l_max, int np, bool plain, bool table_in_smem, const CenterParams& p, unsigned grid,
                        unsigned block, size_t smem, cudaStream_t st);

#define SOAP_DECLARE_L(LV)                                                                                              \
    cudaError_t desc_constants_l##LV(const float* anorm91);                                                             \
    cudaError_t desc_set_smem_l##LV(int np, int bytes);                                                                 \
    cudaError_t desc_launch_l##LV(int np, bool plain, bool table_in_smem, const CenterParams& p, unsigned grid,         \
                                  unsigned block, size_t smem, cudaStream_t st);
SOAP_DECLARE_L(0) SOAP_DECLARE_L(1) SOAP_DECLARE_L(2) SOAP_DECLARE_L(3) SOAP_DECLARE_L(4) SOAP_DECLARE_L(5) SOAP_DECLARE_L(6)
SOAP_DECLARE_L(7) SOAP_DECLARE_L(8) SOAP_DECLARE_L(9) SOAP_DECLARE_L(10) SOAP_DECLARE_L(11) SOAP_DECLARE_L(12)
#undef SOAP_DECLARE_L
}  // namespace soap
