// Reductions over the centres for the averaged output modes.  Both sum in a fixed order, so a
// result does not change from run to run.
#pragma once
#include "soap_device.cuh"

namespace soap {

constexpr int kMeanThreads = 256;
constexpr int kMeanMaxChunks = 128;

// Column sums of in[rows][width] over the rows of chunk blockIdx.y: partial[chunk][width].
__global__ void __launch_bounds__(kMeanThreads)
column_partial_kernel(const float* __restrict__ in, long long rows, int width, long long chunk_rows,
                      double* __restrict__ partial) {
    const int col = blockIdx.x * kMeanThreads + threadIdx.x;
    if (col >= width) return;
    const long long r0 = (long long)blockIdx.y * chunk_rows, r1 = min(rows, r0 + chunk_rows);
    double s = 0.0;
    for (long long r = r0; r < r1; ++r) s += (double)in[r * width + col];
    partial[(size_t)blockIdx.y * width + col] = s;
}

// out[col] = scale * sum over the chunks, in chunk order.
__global__ void __launch_bounds__(kMeanThreads)
column_finish_kernel(const double* __restrict__ partial, int chunks, int width, double scale, float* __restrict__ out) {
    const int col = blockIdx.x * kMeanThreads + threadIdx.x;
    if (col >= width) return;
    double s = 0.0;
    for (int c = 0; c < chunks; ++c) s += partial[(size_t)c * width + col];
    out[col] = (float)(s * scale);
}

// out[j][k][f] = scale * sum over the centres whose row list holds atom j of that row, zero for an
// atom in no list.  CTA (j, slice of the 3 F elements): the threads search the (sorted) row lists of
// 256 centres at a time, compact the hits in centre order and then add the rows up in that order.
constexpr int kAvgThreads = 256;
constexpr int kAvgList = 1024;

__global__ void __launch_bounds__(kAvgThreads)
average_rows_kernel(const float* __restrict__ jac, const long long* __restrict__ row_ptr, const int* __restrict__ row_atom,
                    long long n_centers, int width3, int slice, float scale, float* __restrict__ out) {
    __shared__ long long list[kAvgList];
    __shared__ int warp_cnt[kAvgThreads / 32];
    const int j = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int e0 = blockIdx.y * slice, e1 = min(width3, e0 + slice);
    float* orow = out + (size_t)j * width3;
    int n_list = 0;
    bool first = true;
    auto flush = [&]() {
        __syncthreads();
        for (int e = e0 + tid; e < e1; e += kAvgThreads) {
            float s = 0.f;
            for (int i = 0; i < n_list; ++i) s += jac[(size_t)list[i] * width3 + e];
            if (first) orow[e] = s * scale; else orow[e] += s * scale;
        }
        first = false;
        n_list = 0;
        __syncthreads();
    };
    for (long long c0 = 0; c0 < n_centers; c0 += kAvgThreads) {
        const long long c = c0 + tid;
        long long hit = -1;
        if (c < n_centers) {
            long long lo = row_ptr[c], hi = row_ptr[c + 1];
            while (lo < hi) {
                const long long mid = (lo + hi) >> 1;
                const int a = row_atom[mid];
                if (a == j) { hit = mid; break; }
                if (a < j) lo = mid + 1; else hi = mid;
            }
        }
        const unsigned m = __ballot_sync(0xffffffffu, hit >= 0);
        if (lane == 0) warp_cnt[wid] = __popc(m);
        __syncthreads();
        int before = 0, total = 0;
        for (int w = 0; w < kAvgThreads / 32; ++w) {
            if (w < wid) before += warp_cnt[w];
            total += warp_cnt[w];
        }
        if (n_list + total > kAvgList) flush();                 // uniform over the CTA
        if (hit >= 0) list[n_list + before + __popc(m & ((1u << lane) - 1))] = hit;
        n_list += total;
        __syncthreads();
    }
    flush();
}

}  // namespace soap
