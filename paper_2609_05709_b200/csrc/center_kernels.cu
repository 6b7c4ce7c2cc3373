// Every instantiation of the fused per-centre derivative kernels for one l_max: compiled once per value of
// SOAP_L (0..12), which the build passes on the command line.
#ifndef SOAP_L
#error "compile with -DSOAP_L=<l_max>"
#endif
#include "center_kernel.cuh"
#include "center_launch.h"

namespace soap {

#define SOAP_CAT2(a, b) a##b
#define SOAP_CAT(a, b) SOAP_CAT2(a, b)

template <int KIND, int NM, bool PLAIN>
static cudaError_t set_one(int bytes) {
    return cudaFuncSetAttribute(center_kernel<KIND, SOAP_L, NM, PLAIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}
template <int KIND, int NM, bool PLAIN>
static cudaError_t launch_one(const CenterParams& p, unsigned grid, size_t smem, cudaStream_t st) {
    // the kernel waits on the device for the kernel before it (the row scan, as a rule): its launch and its
    // set-up overlap that kernel's tail
    return launch_dependent(center_kernel<KIND, SOAP_L, NM, PLAIN>, grid, kThreads, smem, st, p);
}

// Fills this translation unit's constant tables (once per process and device is enough;
// it is cheap, so it runs whenever a handle sets up its kernels).
cudaError_t SOAP_CAT(center_constants_l, SOAP_L)(const float* anorm91, const float* dfact16) {
    // norm: (a_lm, (l+m) a_lm);  step: ((2l+1)/(l+1-m), (l+m)/(l+1-m)) for column m and
    // ((2l+1)/(l-m), (l+m+1)/(l-m)) for column m+1 (unused at l = m)
    float2 norm[91];
    float4 step[91];
    for (int l = 0; l <= 12; ++l)
        for (int m = 0; m <= l; ++m) {
            const int t = l * (l + 1) / 2 + m;
            norm[t] = make_float2(anorm91[t], (float)(l + m) * anorm91[t]);
            step[t].x = (float)(2 * l + 1) / (float)(l + 1 - m);
            step[t].y = (float)(l + m) / (float)(l + 1 - m);
            step[t].z = l > m ? (float)(2 * l + 1) / (float)(l - m) : 0.f;
            step[t].w = l > m ? (float)(l + m + 1) / (float)(l - m) : 0.f;
        }
    cudaError_t e = cudaMemcpyToSymbol(kc_norm, norm, sizeof(norm));
    if (e != cudaSuccess) return e;
    e = cudaMemcpyToSymbol(kc_step, step, sizeof(step));
    if (e != cudaSuccess) return e;
    return cudaMemcpyToSymbol(kc_dfact, dfact16, 16 * sizeof(float));
}

// The plain kernels have their own instantiation for the usual n_max (loops over n unroll, the accumulators of
// pass 1 fit the registers exactly; the variant that reads n_max at run time is 1.4 to 2 times slower and
// serves every other n_max); the kernels that honour the options are instantiated for fewer n_max still.
// Even l_max and l_max = 3 get the long lists, the other odd l_max the short ones.
#if (SOAP_L % 2 == 0) || (SOAP_L == 3)
#define SOAP_FOR_FIXED_NMAX(X) X(2) X(4) X(6) X(7) X(8) X(10) X(12)
#define SOAP_FOR_GENERAL_NMAX(X) X(4) X(8)
#else
#define SOAP_FOR_FIXED_NMAX(X) X(4) X(8)
#define SOAP_FOR_GENERAL_NMAX(X) X(8)
#endif
static bool center_has_fixed_nmax(int n_max) {
    switch (n_max) {
#define X(N) case N: return true;
        SOAP_FOR_FIXED_NMAX(X)
#undef X
    }
    return false;
}
static bool general_has_fixed_nmax(int n_max) {
    switch (n_max) {
#define X(N) case N: return true;
        SOAP_FOR_GENERAL_NMAX(X)
#undef X
    }
    return false;
}

cudaError_t SOAP_CAT(center_set_smem_l, SOAP_L)(int kind, int n_max, int bytes) {
    cudaError_t e;
    if (kind == kCenterInner) {
        if ((e = set_one<3, 0, false>(bytes)) != cudaSuccess) return e;
        return set_one<3, 8, false>(bytes);
    }
    if (kind == kCenterOuter) {
        if ((e = set_one<4, 0, false>(bytes)) != cudaSuccess) return e;
        return set_one<4, 8, false>(bytes);
    }
    if (kind == kCenterCoeff) {
        if ((e = set_one<2, 0, false>(bytes)) != cudaSuccess) return e;
        switch (general_has_fixed_nmax(n_max) ? n_max : 0) {
#define X(N) case N: return set_one<2, N, false>(bytes);
            SOAP_FOR_GENERAL_NMAX(X)
#undef X
        }
        return cudaSuccess;
    }
    if ((e = set_one<1, 0, false>(bytes)) != cudaSuccess) return e;
    switch (general_has_fixed_nmax(n_max) ? n_max : 0) {
#define X(N) case N: e = set_one<1, N, false>(bytes); break;
        SOAP_FOR_GENERAL_NMAX(X)
#undef X
        default: e = cudaSuccess;
    }
    if (e != cudaSuccess) return e;
    switch (center_has_fixed_nmax(n_max) ? n_max : 0) {
#define X(N) case N: return set_one<1, N, true>(bytes);
        SOAP_FOR_FIXED_NMAX(X)
#undef X
        default: return set_one<1, 0, true>(bytes);
    }
}

cudaError_t SOAP_CAT(center_launch_l, SOAP_L)(int kind, int n_max, bool plain, const CenterParams& p, unsigned grid, size_t smem,
                                              cudaStream_t st) {
    if (kind == kCenterInner)
        return n_max == 8 ? launch_one<3, 8, false>(p, grid, smem, st) : launch_one<3, 0, false>(p, grid, smem, st);
    if (kind == kCenterOuter)
        return n_max == 8 ? launch_one<4, 8, false>(p, grid, smem, st) : launch_one<4, 0, false>(p, grid, smem, st);
    if (kind == kCenterCoeff) {
        switch (general_has_fixed_nmax(n_max) ? n_max : 0) {
#define X(N) case N: return launch_one<2, N, false>(p, grid, smem, st);
            SOAP_FOR_GENERAL_NMAX(X)
#undef X
            default: return launch_one<2, 0, false>(p, grid, smem, st);
        }
    }
    if (!plain) {
        switch (general_has_fixed_nmax(n_max) ? n_max : 0) {
#define X(N) case N: return launch_one<1, N, false>(p, grid, smem, st);
            SOAP_FOR_GENERAL_NMAX(X)
#undef X
            default: return launch_one<1, 0, false>(p, grid, smem, st);
        }
    }
    switch (center_has_fixed_nmax(n_max) ? n_max : 0) {
#define X(N) case N: return launch_one<1, N, true>(p, grid, smem, st);
        SOAP_FOR_FIXED_NMAX(X)
#undef X
        default: return launch_one<1, 0, true>(p, grid, smem, st);
    }
}

}  // namespace soap
