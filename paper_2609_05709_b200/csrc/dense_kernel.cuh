// Dense view of the neighbour-sparse Jacobian: out[c][a][3][F] for the atoms of an inclusion
// list (the layout the paper's derivatives() returns; every entry outside a centre's sphere is an
// explicit zero).  One CTA per (centre, listed atom): a binary search in the centre's ascending
// row_atom segment finds the row, which is copied, or zeros are written.  Pure HBM traffic.
#pragma once
#include "soap_device.cuh"

namespace soap {

__global__ void __launch_bounds__(128)
dense_scatter_kernel(const float* __restrict__ jac_rows, const long long* __restrict__ row_ptr,
                     const int* __restrict__ row_atom, long long n_centers, const int* __restrict__ include,
                     long long n_include, int F, float* __restrict__ out) {
    const long long slot = blockIdx.x;                      // c * n_include + a
    const long long c = slot / n_include, a = slot - c * n_include;
    const int atom = include ? include[a] : (int)a;
    long long lo = row_ptr[c], hi = row_ptr[c + 1];         // first row with row_atom >= atom
    while (lo < hi) {
        const long long mid = (lo + hi) >> 1;
        if (row_atom[mid] < atom) lo = mid + 1; else hi = mid;
    }
    const bool found = lo < row_ptr[c + 1] && row_atom[lo] == atom;
    const float* src = jac_rows + (size_t)lo * 3 * F;
    float* dst = out + (size_t)slot * 3 * F;
    for (int e = threadIdx.x; e < 3 * F; e += blockDim.x) dst[e] = found ? src[e] : 0.f;
}

// Species-compact rows back to full rows: out[r][3][F].  One CTA per centre walks the centre's
// rows; a neighbour's compact row is scattered through the column map of its species (zeros
// elsewhere), the centre's own row is copied from its separate array.
__global__ void __launch_bounds__(256)
compact_expand_kernel(const float* __restrict__ jac_compact, const float* __restrict__ center_rows,
                      const long long* __restrict__ row_ptr, const int* __restrict__ row_atom,
                      const int* __restrict__ centers, const int* __restrict__ numbers, const int* __restrict__ zlut,
                      const int* __restrict__ col_map, int n_compact, int pitch, int F, float* __restrict__ out) {
    const long long c = blockIdx.x;
    const int ci = centers ? centers[c] : (int)c;
    for (long long r = row_ptr[c]; r < row_ptr[c + 1]; ++r) {
        float* dst = out + (size_t)r * 3 * F;
        const int atom = row_atom[r];
        if (atom == ci) {
            const float* src = center_rows + (size_t)c * 3 * F;
            for (int e = threadIdx.x; e < 3 * F; e += blockDim.x) dst[e] = src[e];
            continue;
        }
        for (int e = threadIdx.x; e < 3 * F; e += blockDim.x) dst[e] = 0.f;
        __syncthreads();
        const int z = zlut[numbers[atom]];
        const int* map = col_map + (size_t)z * n_compact;
        const float* src = jac_compact + (size_t)r * 3 * pitch;
        for (int e = threadIdx.x; e < 3 * n_compact; e += blockDim.x) {
            const int k = e / n_compact, j = e - k * n_compact;
            dst[(size_t)k * F + map[j]] = src[(size_t)k * pitch + j];
        }
        __syncthreads();
    }
}

}  // namespace soap
