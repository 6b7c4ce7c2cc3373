// Dispatch of the per-centre kernel over its compile-time l_max (0..12) and n_max.
#pragma once
#include "soap_device.cuh"

namespace soap {
// kernel kinds: descriptor and Jacobian; coefficients c^mu_nlm and their Jacobian; Jacobian of the inner average;
// Jacobian of the outer average (the last two: every atom a centre, one row per atom)
constexpr int kCenterDeriv = 1, kCenterCoeff = 2, kCenterInner = 3, kCenterOuter = 4;
// whether the parameters ask for nothing beyond the default configuration (the kernels instantiated with
// PLAIN = true assume exactly this)
inline bool center_params_plain(const CenterParams& p) {
    return p.crossover && !p.compact && !p.emit_coeff && !p.c_bar && !p.sites && !p.pair_w && p.w0 == 1.f && !p.inner_rows && !p.c_all;
}
// harmonic tables up to l = 12: anorm[91] (index l(l+1)/2 + m), dfact[16]
cudaError_t center_constants(int l_max, const float* anorm91, const float* dfact16);
cudaError_t center_set_smem(int kind, int l_max, int n_max, int bytes);
cudaError_t center_launch(int kind, int l_max, int n_max, const CenterParams& p, unsigned grid, size_t smem, cudaStream_t st);

#define SOAP_DECLARE_L(LV)                                                                                       \
    cudaError_t center_constants_l##LV(const float* anorm91, const float* dfact16);         \
    cudaError_t center_set_smem_l##LV(int kind, int n_max, int bytes);                                        \
    cudaError_t center_launch_l##LV(int kind, int n_max, bool plain, const CenterParams& p, unsigned grid, size_t smem, cudaStream_t st);
SOAP_DECLARE_L(0) SOAP_DECLARE_L(1) SOAP_DECLARE_L(2) SOAP_DECLARE_L(3) SOAP_DECLARE_L(4) SOAP_DECLARE_L(5) SOAP_DECLARE_L(6)
SOAP_DECLARE_L(7) SOAP_DECLARE_L(8) SOAP_DECLARE_L(9) SOAP_DECLARE_L(10) SOAP_DECLARE_L(11) SOAP_DECLARE_L(12)
#undef SOAP_DECLARE_L
}  // namespace soap
