// Every instantiation of the descriptor-only kernel for one l_max: compiled once per value of SOAP_L (0..12),
// which the build passes on the command line.
#ifndef SOAP_L
#error "compile with -DSOAP_L=<l_max>"
#endif
#include "desc_kernel.cuh"
#include "desc_launch.h"

namespace soap {

#define SOAP_CAT2(a, b) a##b
#define SOAP_CAT(a, b) SOAP_CAT2(a, b)

// the default configuration runs with the table in shared memory or in global memory; calls that use an option
// always read the table from global memory
#define SOAP_DESC_VARIANTS(X, NP) X(NP, true, true) X(NP, true, false) X(NP, false, false)

template <int NP>
static cudaError_t set_np(int bytes) {
    cudaError_t e = cudaSuccess;
#define X(N, PL, TS)                                                                                                        \
    if (e == cudaSuccess) e = cudaFuncSetAttribute(desc_kernel<SOAP_L, N, PL, TS>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    SOAP_DESC_VARIANTS(X, NP)
#undef X
    return e;
}

template <int NP>
static cudaError_t launch_np(bool plain, bool ts, const CenterParams& p, unsigned grid, unsigned block, size_t smem, cudaStream_t st) {
    // (the kernel waits on the device for the kernel before it: launch and table staging overlap that kernel's tail)
    if (plain && ts) return launch_dependent(desc_kernel<SOAP_L, NP, true, true>, grid, block, smem, st, p);
    if (plain) return launch_dependent(desc_kernel<SOAP_L, NP, true, false>, grid, block, smem, st, p);
    return launch_dependent(desc_kernel<SOAP_L, NP, false, false>, grid, block, smem, st, p);
}

cudaError_t SOAP_CAT(desc_constants_l, SOAP_L)(const float* anorm91) {
    return cudaMemcpyToSymbol(kd_norm, anorm91, 91 * sizeof(float));
}

cudaError_t SOAP_CAT(desc_set_smem_l, SOAP_L)(int np, int bytes) {
    switch (np) {
        case 4: return set_np<4>(bytes);
        case 8: return set_np<8>(bytes);
        case 12: return set_np<12>(bytes);
        case 16: return set_np<16>(bytes);
    }
    return cudaErrorInvalidValue;
}

cudaError_t SOAP_CAT(desc_launch_l, SOAP_L)(int np, bool plain, bool ts, const CenterParams& p, unsigned grid, unsigned block,
                                            size_t smem, cudaStream_t st) {
    switch (np) {
        case 4: return launch_np<4>(plain, ts, p, grid, block, smem, st);
        case 8: return launch_np<8>(plain, ts, p, grid, block, smem, st);
        case 12: return launch_np<12>(plain, ts, p, grid, block, smem, st);
        case 16: return launch_np<16>(plain, ts, p, grid, block, smem, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace soap
