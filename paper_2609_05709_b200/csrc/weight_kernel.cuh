// Radial weighting of the neighbour density: w(d) and w'(d)/d of every pair, in fp64, written once per
// neighbour search so that the fused per-centre kernel only multiplies.  The paper names the option
// and no formula; the forms below are the reading stated with soap_set_weighting.
#pragma once
#include "soap_device.cuh"

namespace soap {

struct WeightParams {
    int fn;                       // 0 none, 1 poly, 2 pow, 3 exp
    double r0, c, d, m;
};

__device__ inline void weight_eval(const WeightParams& wp, double dist, double& w, double& dw) {
    const double x = dist / wp.r0;
    if (wp.fn == 1) {
        // c (1 + 2 x^3 - 3 x^2)^m inside r0, zero outside
        const double base = 1.0 + x * x * (2.0 * x - 3.0);
        if (x <= 1.0 && base > 0.0) {
            w = wp.c * pow(base, wp.m);
            dw = wp.c * wp.m * pow(base, wp.m - 1.0) * (6.0 * x * x - 6.0 * x) / wp.r0;
        } else {
            w = (x <= 1.0 && wp.m == 0.0) ? wp.c : 0.0;
            dw = 0.0;
        }
    } else if (wp.fn == 2) {
        // c / (d + x^m)
        const double pw = pow(x, wp.m), den = wp.d + pw;
        w = wp.c / den;
        dw = -wp.c * (wp.m * pw / dist) / (den * den);
    } else {
        // c / (d + exp(-x))
        const double e = exp(-x), den = wp.d + e;
        w = wp.c / den;
        dw = wp.c * e / wp.r0 / (den * den);
    }
}

// One warp per centre walks the centre's pair segment.  The displacement is formed exactly as in
// the per-centre kernel.
__global__ void __launch_bounds__(256)
pair_weight_kernel(const float* __restrict__ pos, const int* __restrict__ centers, const float* __restrict__ sites,
                   long long n_centers, Geometry geom,
                   const long long* __restrict__ pair_start, const int* __restrict__ pair_count,
                   const unsigned long long* __restrict__ pair_key, long long pair_capacity, const Counters* counters,
                   WeightParams wp, float2* __restrict__ pair_w) {
    if (counters->n_pairs > pair_capacity) return;            // failed build: the segments are not there
    const long long c_idx = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (c_idx >= n_centers) return;
    const int lane = threadIdx.x & 31;
    const int ci = centers ? centers[c_idx] : (int)c_idx;
    const float* pc = sites ? sites + 3 * c_idx : pos + 3 * (long long)ci;
    const float xi = pc[0], yi = pc[1], zi = pc[2];
    const long long base = pair_start[c_idx];
    const int k = pair_count[c_idx];
    const bool periodic = geom.pbc[0] | geom.pbc[1] | geom.pbc[2];
    for (int e = lane; e < k; e += 32) {
        const unsigned long long key = pair_key[base + e];
        const int j = key_atom(key);
        double dx = (double)pos[3 * (long long)j] - (double)xi;
        double dy = (double)pos[3 * (long long)j + 1] - (double)yi;
        double dz = (double)pos[3 * (long long)j + 2] - (double)zi;
        if (periodic) {
            int s[3];
            key_shift(key, s);
            dx += s[0] * geom.cell[0] + s[1] * geom.cell[3] + s[2] * geom.cell[6];
            dy += s[0] * geom.cell[1] + s[1] * geom.cell[4] + s[2] * geom.cell[7];
            dz += s[0] * geom.cell[2] + s[1] * geom.cell[5] + s[2] * geom.cell[8];
        }
        const double r = sqrt(dx * dx + dy * dy + dz * dz);
        double w, dw;
        weight_eval(wp, r, w, dw);
        pair_w[base + e] = make_float2((float)w, (float)(dw / r));
    }
}

}  // namespace soap
