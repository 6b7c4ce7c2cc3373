// C ABI of libsoap_b200: handle, scratch memory and the launch sequences.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "basis_host.h"
#include "average_kernels.cuh"
#include "center_launch.h"
#include "dense_kernel.cuh"
#include "desc_kernel.cuh"
#include "desc_launch.h"
#include "neighbor_kernels.cuh"
#include "soap.h"
#include "weight_kernel.cuh"

using namespace soap;

namespace soap {
cudaError_t center_constants(int l_max, const float* anorm91, const float* dfact16) {
    switch (l_max) {
#define X(LV) case LV: return center_constants_l##LV(anorm91, dfact16);
        X(0) X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8) X(9) X(10) X(11) X(12)
#undef X
    }
    return cudaErrorInvalidValue;
}
cudaError_t center_set_smem(int kind, int l_max, int n_max, int bytes) {
    switch (l_max) {
#define X(LV) case LV: return center_set_smem_l##LV(kind, n_max, bytes);
        X(0) X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8) X(9) X(10) X(11) X(12)
#undef X
    }
    return cudaErrorInvalidValue;
}
cudaError_t center_launch(int kind, int l_max, int n_max, const CenterParams& p, unsigned grid, size_t smem, cudaStream_t st) {
    switch (l_max) {
#define X(LV) case LV: return center_launch_l##LV(kind, n_max, center_params_plain(p), p, grid, smem, st);
        X(0) X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8) X(9) X(10) X(11) X(12)
#undef X
    }
    return cudaErrorInvalidValue;
}
cudaError_t desc_constants(int l_max, const float* anorm91) {
    switch (l_max) {
#define X(LV) case LV: return desc_constants_l##LV(anorm91);
        X(0) X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8) X(9) X(10) X(11) X(12)
#undef X
    }
    return cudaErrorInvalidValue;
}
cudaError_t desc_set_smem(int l_max, int np, int bytes) {
    switch (l_max) {
#define X(LV) case LV: return desc_set_smem_l##LV(np, bytes);
        X(0) X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8) X(9) X(10) X(11) X(12)
#undef X
    }
    return cudaErrorInvalidValue;
}
cudaError_t desc_launch(int l_max, int np, bool plain, bool table_in_smem, const CenterParams& p, unsigned grid, unsigned block,
                        size_t smem, cudaStream_t st) {
    switch (l_max) {
#define X(LV) case LV: return desc_launch_l##LV(np, plain, table_in_smem, p, grid, block, smem, st);
        X(0) X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8) X(9) X(10) X(11) X(12)
#undef X
    }
    return cudaErrorInvalidValue;
}
}  // namespace soap

struct soap_handle {
    // configuration
    std::vector<int> species;            // sorted atomic numbers
    int S = 0, n_max = 0, l_max = 0, rbf = 0;
    double r_cut = 0, sigma = 0;
    int pbc[3] = {0, 0, 0};
    int crossover = 1;
    WeightParams weight = {0, 1.0, 1.0, 1.0, 1.0};   // radial weighting of the neighbour density (off)
    double w0 = 1.0;
    int64_t F = 0;
    HostBasis basis;
    std::vector<int> feat_pack;
    std::vector<int> compact_map;        // [S][Fc] full feature index of each column of a species-compact row
    int64_t Fc = 0, Fc_pitch = 0;
    int* d_compact_map = nullptr;
    std::string error;
    // device state (created on first use)
    int device = -1;
    bool tables_ready = false;
    float *d_table = nullptr, *d_self = nullptr, *d_kl = nullptr;
    float* d_table_ln = nullptr;         // the radial table re-laid for the descriptor-only kernel
    int sm_count = 0, max_smem = 0;
    int desc_np = 0;                     // n_max rounded up to a multiple of four
    size_t desc_table_bytes = 0, desc_warp_bytes = 0;
    int *d_feat = nullptr, *d_zlut = nullptr, *d_l_of_lm = nullptr;
    Counters* d_counters = nullptr;
    unsigned long long* d_bbox = nullptr;   // 6 words of bounding box (structures above 16384 atoms)
    int* d_order = nullptr;
    GridParams* d_grid = nullptr;
    Counters* h_counters = nullptr;      // pinned
    // scratch, grown on demand
    int64_t cap_atoms = 0, cap_centers = 0, cap_cells = 0, cap_pairs = 0;
    int *d_species_idx = nullptr, *d_atom_cell = nullptr, *d_atom_wrap = nullptr, *d_s_wrap = nullptr;
    float4* d_s_pos = nullptr;
    int *d_cell_count = nullptr, *d_cell_start = nullptr;
    int *d_pair_count = nullptr, *d_row_count = nullptr, *d_self_row = nullptr;
    long long *d_pair_ptr = nullptr, *d_pair_start = nullptr, *d_row_ptr = nullptr, *d_tile_offsets = nullptr;
    int *d_tile_sums = nullptr, *d_cell_tile_sums = nullptr;
    long long* d_cell_tile_offsets = nullptr;
    unsigned long long *d_pair_key = nullptr, *d_pair_tmp = nullptr;
    int* d_pair_row = nullptr;
    float2* d_pair_w = nullptr;          // per-pair weights, only with a radial weighting
    void* d_work = nullptr;              // workspace of the averaged modes
    size_t cap_work = 0;
    // plan
    int64_t planned_atoms = -1, planned_centers = -1;
    int64_t pairs_per_center_hint = 0;   // average at the last plan (chooses the pair kernel variant)
    int64_t last_centers = 0;
    bool list_sorted = false;            // whether the pair list of the last search is sorted (descriptor-only calls skip that)
    int P_deriv = 16, P_outer = 16;      // pairs per staged chunk: derivative kernels, kernel of the outer average
    size_t smem_deriv = 0, smem_outer = 0;
    bool outer_fast = false;             // whether the kernel of the outer average fits the shared memory
    // optional per-segment timing (events on the caller's stream)
    bool profiling = false;
    cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};
};

namespace {

constexpr int64_t kOrderMaxCenters = 65536;   // above this the CTAs simply run in centre order

int fail(soap_t* h, int code, const std::string& msg) {
    if (h) h->error = msg;
    return code;
}
int cuda_fail(soap_t* h, cudaError_t e, const char* what) {
    return fail(h, SOAP_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}
#define CU(call)                                                   \
    do {                                                           \
        cudaError_t e_ = (call);                                   \
        if (e_ != cudaSuccess) return cuda_fail(h, e_, #call);     \
    } while (0)

template <typename T>
cudaError_t upload(T** dst, const std::vector<T>& src) {
    cudaError_t e = cudaMalloc((void**)dst, std::max<size_t>(src.size(), 1) * sizeof(T));
    if (e != cudaSuccess) return e;
    return cudaMemcpy(*dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice);
}

template <typename T>
cudaError_t regrow(T** ptr, size_t count) {
    if (*ptr) { cudaFree(*ptr); *ptr = nullptr; }
    return cudaMalloc((void**)ptr, std::max<size_t>(count, 1) * sizeof(T));
}

bool invert3(const double m[9], double inv[9], double& det) {
    det = m[0] * (m[4] * m[8] - m[5] * m[7]) - m[1] * (m[3] * m[8] - m[5] * m[6]) + m[2] * (m[3] * m[7] - m[4] * m[6]);
    if (!(std::fabs(det) > 1e-12)) return false;
    inv[0] = (m[4] * m[8] - m[5] * m[7]) / det; inv[1] = (m[2] * m[7] - m[1] * m[8]) / det; inv[2] = (m[1] * m[5] - m[2] * m[4]) / det;
    inv[3] = (m[5] * m[6] - m[3] * m[8]) / det; inv[4] = (m[0] * m[8] - m[2] * m[6]) / det; inv[5] = (m[2] * m[3] - m[0] * m[5]) / det;
    inv[6] = (m[3] * m[7] - m[4] * m[6]) / det; inv[7] = (m[1] * m[6] - m[0] * m[7]) / det; inv[8] = (m[0] * m[4] - m[1] * m[3]) / det;
    return true;
}

int make_geometry(soap_t* h, const double* cell, Geometry& g) {
    const bool periodic = h->pbc[0] || h->pbc[1] || h->pbc[2];
    if (periodic && !cell) return fail(h, SOAP_ERR_INVALID_ARG, "a periodic axis needs a cell");
    static const double ident[9] = {1, 0, 0, 0, 1, 0, 0, 0, 1};
    std::memcpy(g.cell, cell ? cell : ident, sizeof(g.cell));
    double det;
    if (!invert3(g.cell, g.inv, det)) return fail(h, SOAP_ERR_INVALID_ARG, "the cell is singular");
    for (int a = 0; a < 3; ++a) {
        const double* u = &g.cell[3 * ((a + 1) % 3)];
        const double* v = &g.cell[3 * ((a + 2) % 3)];
        double cx = u[1] * v[2] - u[2] * v[1], cy = u[2] * v[0] - u[0] * v[2], cz = u[0] * v[1] - u[1] * v[0];
        g.height[a] = std::fabs(det) / std::sqrt(cx * cx + cy * cy + cz * cz);
        g.pbc[a] = h->pbc[a];
        if (h->pbc[a] && std::ceil(h->r_cut / g.height[a]) > 100)
            return fail(h, SOAP_ERR_INVALID_ARG, "the cell is too thin for this cutoff (more than 100 images along an axis)");
    }
    g.r_cut = h->r_cut;
    g.rc2 = h->r_cut * h->r_cut;
    return SOAP_OK;
}

// Shared-memory plan of the per-centre kernels (depends on the basis and on whether pairs carry weights).
int plan_smem(soap_t* h) {
    // shared-memory plan of the per-centre kernels
    int max_smem = 0;
    CU(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, h->device));
    h->max_smem = max_smem;
    h->desc_warp_bytes = (size_t)make_desc_layout(h->S, desc_np(h->n_max), h->l_max, 1, 0).per_warp * 4;
    if (h->desc_warp_bytes > (size_t)max_smem) return fail(h, SOAP_ERR_INVALID_ARG, "this basis does not fit the shared memory of the device");
    CU(desc_set_smem(h->l_max, desc_np(h->n_max), max_smem));
    // pairs per staged chunk of the derivative kernels: the largest that still leaves room for three CTAs per SM,
    // else two, else whatever fits (`extra` bytes follow the usual layout); false if nothing fits
    auto plan_chunk = [&](size_t extra, int& P_out, size_t& bytes_out) -> bool {
        int P = 32;
        size_t bytes = 0;
        const size_t budget3 = (size_t)228 * 1024 / 3 - 1024, budget2 = (size_t)228 * 1024 / 2 - 1024;
        for (int pass = 0; pass < 3; ++pass) {
            const size_t budget = pass == 0 ? budget3 : pass == 1 ? budget2 : (size_t)max_smem;
            for (P = 32; P >= 4; P /= 2) {
                bytes = (size_t)make_layout(h->S, h->n_max, h->l_max, P, true, h->weight.fn != 0).total * 4 + extra;
                if (bytes <= budget) break;
            }
            if (P >= (pass == 2 ? 4 : 8) && bytes <= budget) break;
            if (P < 4) P = 4;
        }
        bytes = (size_t)make_layout(h->S, h->n_max, h->l_max, P, true, h->weight.fn != 0).total * 4 + extra;
        P_out = P; bytes_out = bytes;
        return bytes <= (size_t)max_smem;
    };
    if (!plan_chunk(0, h->P_deriv, h->smem_deriv)) return fail(h, SOAP_ERR_INVALID_ARG, "this basis does not fit the shared memory of the device");
    CU(center_set_smem(kCenterDeriv, h->l_max, h->n_max, (int)h->smem_deriv));
    CU(center_set_smem(kCenterCoeff, h->l_max, h->n_max, (int)h->smem_deriv));
    CU(center_set_smem(kCenterInner, h->l_max, h->n_max, (int)h->smem_deriv));
    // the kernel of the outer average keeps, per warp, a copy of a neighbouring centre's coefficients behind the usual
    // layout; a basis too large for that takes the general path (per-pair rows in a workspace)
    const int LMP = ((h->l_max + 1) * (h->l_max + 1)) | 1;
    h->outer_fast = plan_chunk((size_t)kWarps * h->S * h->n_max * LMP * 4, h->P_outer, h->smem_outer);
    if (h->outer_fast) CU(center_set_smem(kCenterOuter, h->l_max, h->n_max, (int)h->smem_outer));
    return SOAP_OK;
}

int ensure_device(soap_t* h) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(h, e, "cudaGetDevice (is a CUDA device present? this library has no CPU path)");
    if (h->tables_ready) {
        if (dev != h->device) return fail(h, SOAP_ERR_INVALID_ARG, "handle was first used on another device");
        return SOAP_OK;
    }
    h->device = dev;
    CU(upload(&h->d_table, h->basis.table));
    {
        // [interval][l][n / 2][6][2], n padded to a multiple of four: the coefficients of two adjacent n interleaved
        // (the descriptor-only kernel evaluates them with packed multiply-adds); the padding channels are zero
        const int L1 = h->l_max + 1, n_ch = h->n_max * L1, np = desc_np(h->n_max);
        std::vector<float> ln((size_t)h->basis.n_intervals_values * L1 * np * kTableCoef, 0.f);
        for (int q = 0; q < h->basis.n_intervals_values; ++q)
            for (int l = 0; l < L1; ++l)
                for (int n = 0; n < h->n_max; ++n)
                    for (int k = 0; k < kTableCoef; ++k)
                        ln[((((size_t)q * L1 + l) * (np / 2) + n / 2) * kTableCoef + k) * 2 + (n & 1)] =
                            h->basis.table_values[((size_t)q * n_ch + n * L1 + l) * kTableCoef + k];
        CU(upload(&h->d_table_ln, ln));
        h->desc_np = np;
        h->desc_table_bytes = ln.size() * sizeof(float);
    }
    CU(cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device));
    CU(upload(&h->d_self, h->basis.self_term));
    CU(upload(&h->d_kl, h->basis.kl));
    CU(upload(&h->d_feat, h->feat_pack));
    {
        std::vector<int> l_of_lm;
        for (int l = 0; l <= h->l_max; ++l)
            for (int m = -l; m <= l; ++m) l_of_lm.push_back(l);
        CU(upload(&h->d_l_of_lm, l_of_lm));
    }
    std::vector<int> lut(128, -1);
    for (int s = 0; s < h->S; ++s) lut[h->species[s]] = s;
    CU(upload(&h->d_zlut, lut));
    CU(cudaMalloc((void**)&h->d_counters, sizeof(Counters)));
    CU(cudaMemset(h->d_counters, 0, sizeof(Counters)));
    CU(cudaMalloc((void**)&h->d_bbox, 64));
    CU(cudaMalloc((void**)&h->d_grid, sizeof(GridParams)));
    CU(cudaMallocHost((void**)&h->h_counters, sizeof(Counters)));
    if (int rc = plan_smem(h)) return rc;
    {
        // universal harmonic tables up to l = 12 (the handle's own tables stop at its l_max)
        std::vector<float> anorm(91, 0.f), dfact(16, 0.f);
        for (size_t i = 0; i < h->basis.anorm.size(); ++i) anorm[i] = h->basis.anorm[i];
        for (size_t i = 0; i < h->basis.dfact.size(); ++i) dfact[i] = h->basis.dfact[i];
        CU(center_constants(h->l_max, anorm.data(), dfact.data()));
        CU(desc_constants(h->l_max, anorm.data()));
    }
    h->tables_ready = true;
    return SOAP_OK;
}

int ensure_scratch(soap_t* h, int64_t N, int64_t C, int64_t pairs) {
    if (N > h->cap_atoms || h->cap_atoms == 0) {
        int64_t cap = N + N / 8 + 256;
        CU(regrow(&h->d_species_idx, cap));
        CU(regrow(&h->d_atom_cell, cap));
        CU(regrow(&h->d_atom_wrap, cap));
        CU(regrow(&h->d_s_wrap, cap));
        CU(regrow(&h->d_s_pos, cap));
        int64_t cells = std::min<int64_t>(std::max<int64_t>(2 * cap, 4096), (int64_t)1 << 26);
        CU(regrow(&h->d_cell_count, cells + 1));
        CU(regrow(&h->d_cell_start, cells + 1));
        CU(regrow(&h->d_cell_tile_sums, cells / kScanTile + 2));
        CU(regrow(&h->d_cell_tile_offsets, cells / kScanTile + 3));
        h->cap_cells = cells;
        h->cap_atoms = cap;
    }
    if (C > h->cap_centers || h->cap_centers == 0) {
        int64_t cap = C + C / 8 + 256;
        CU(regrow(&h->d_pair_count, cap));
        CU(regrow(&h->d_row_count, cap));
        CU(regrow(&h->d_self_row, cap));
        CU(regrow(&h->d_order, cap));
        CU(regrow(&h->d_pair_ptr, cap + 1));
        CU(regrow(&h->d_pair_start, cap));
        CU(regrow(&h->d_row_ptr, cap + 1));
        CU(regrow(&h->d_tile_sums, cap / kScanTile + 2));
        CU(regrow(&h->d_tile_offsets, cap / kScanTile + 3));
        h->cap_centers = cap;
    }
    if (pairs > h->cap_pairs || h->cap_pairs == 0) {
        int64_t cap = pairs + pairs / 4 + 1024;
        CU(regrow(&h->d_pair_key, cap));
        CU(regrow(&h->d_pair_tmp, cap));
        CU(regrow(&h->d_pair_row, cap));
        if (h->weight.fn) CU(regrow(&h->d_pair_w, cap));
        h->cap_pairs = cap;
    }
    return SOAP_OK;
}

int blocks_for(int64_t n, int threads, int cap = 4096) {
    return (int)std::max<int64_t>(1, std::min<int64_t>((n + threads - 1) / threads, cap));
}

// Exclusive scan of C per-centre counts into out[0..C] (out[C] = total, also to *total_dev).
void scan_counts(soap_t* h, const int* counts, long long* out, int64_t C, long long* total_dev, cudaStream_t st) {
    if (C <= 65536) {
        scan_kernel<long long><<<1, 1024, 0, st>>>(counts, out, C, total_dev);
        return;
    }
    const long long tiles = (C + kScanTile - 1) / kScanTile;
    tile_sum_kernel<<<(unsigned)tiles, 1024, 0, st>>>(counts, C, h->d_tile_sums);
    scan_kernel<long long><<<1, 1024, 0, st>>>(h->d_tile_sums, h->d_tile_offsets, tiles, total_dev);
    tile_scan_kernel<long long><<<(unsigned)tiles, 1024, 0, st>>>(counts, out, C, h->d_tile_offsets, tiles);
}

// The whole neighbour search: cell list, sorted pair segments with their row bookkeeping, row
// pointers (to `row_ptr_out`, the caller's array or the handle's) and the launch order.
// With `batch` (struct_ptr [n_structs+1], device): many independent non-periodic structures in one list of atoms,
// every atom a centre, neighbours only inside the own structure.
struct Batch {
    const long long* struct_ptr = nullptr;
    int64_t n_structs = 0;
};
// A single small non-periodic structure with every atom a centre takes the same brute-force pair kernel (one
// launch instead of the two that build and walk a cell list).
constexpr int64_t kBruteForceAtoms = 512;

int launch_neighbors(soap_t* h, const float* pos, const int32_t* num, int64_t N, const Geometry& g,
                     const int32_t* centers, const float* sites, int64_t C, long long* row_ptr_out, cudaStream_t st,
                     const Batch& batch = Batch(), bool rows = true) {
    // (C == N: the brute-force kernel writes the per-centre arrays for every atom, and those are sized from C)
    const bool brute = !batch.struct_ptr && !centers && !sites && C == N && N <= kBruteForceAtoms && !(g.pbc[0] | g.pbc[1] | g.pbc[2]);
    if (batch.struct_ptr || brute) {
        CU(cudaMemsetAsync(&h->d_counters->n_pairs, 0, 2 * sizeof(long long), st));      // pair cursor and row total
        if (N > 0) batch_pairs_kernel<<<(unsigned)((N + kFillWarps - 1) / kFillWarps), kFillWarps * 32, 0, st>>>(
            pos, num, h->d_zlut, h->d_species_idx, batch.struct_ptr, batch.n_structs, N, g.rc2, h->cap_pairs, h->d_pair_key,
            h->d_pair_row, h->d_pair_start, h->d_pair_count, h->d_row_count, h->d_self_row, h->d_counters);
    } else if (N <= kSmallPrepAtoms) {
        small_prep_kernel<<<1, kPrepThreads, 0, st>>>(pos, num, N, g, h->d_zlut, h->d_species_idx, (int)h->cap_cells, h->d_grid,
                                                      h->d_atom_cell, h->d_atom_wrap, h->d_cell_count, h->d_cell_start,
                                                      h->d_s_pos, h->d_s_wrap, h->d_counters);
    } else {
        CU(cudaMemsetAsync(h->d_bbox, 0, 64, st));
        CU(cudaMemsetAsync(h->d_cell_count, 0, (h->cap_cells + 1) * sizeof(int), st));
        species_bbox_kernel<<<blocks_for(N, 256, 1024), 256, 0, st>>>(pos, num, N, g, h->d_zlut, h->d_species_idx, h->d_bbox, h->d_counters);
        grid_setup_kernel<<<1, 1, 0, st>>>(h->d_bbox, g, N, (int)h->cap_cells, h->d_grid, h->d_counters);
        bin_count_kernel<<<blocks_for(N, 256), 256, 0, st>>>(pos, N, g, h->d_grid, h->d_atom_cell, h->d_atom_wrap, h->d_cell_count, h->d_counters);
        {
            // exclusive scan of the bin counts over the whole (zero-filled) capacity, tile by tile
            const long long tiles = (h->cap_cells + kScanTile - 1) / kScanTile;
            tile_sum_kernel<<<(unsigned)tiles, 1024, 0, st>>>(h->d_cell_count, h->cap_cells, h->d_cell_tile_sums);
            scan_kernel<long long><<<1, 1024, 0, st>>>(h->d_cell_tile_sums, h->d_cell_tile_offsets, tiles, nullptr);
            tile_scan_kernel<int><<<(unsigned)tiles, 1024, 0, st>>>(h->d_cell_count, h->d_cell_start, h->cap_cells, h->d_cell_tile_offsets, tiles);
        }
        bin_fill_kernel<<<blocks_for(N, 256), 256, 0, st>>>(pos, N, h->d_atom_cell, h->d_atom_wrap, h->d_cell_start, h->d_cell_count, h->d_s_pos, h->d_s_wrap);
    }
    if (C > 0 && !batch.struct_ptr && !brute) {
        // few pairs per centre at the last plan: the variant with the small on-chip key buffers (more warps resident);
        // descriptor-only calls take the variants without sorting and row bookkeeping
        const bool small_keys = h->pairs_per_center_hint > 0 && h->pairs_per_center_hint <= kFillSmemKeysSmall * 3 / 4;
        const unsigned grid = (unsigned)((C + kFillWarps - 1) / kFillWarps);
#define SOAP_PAIRS_ARGS pos, centers, sites, C, g, h->d_grid, h->d_atom_cell, h->d_atom_wrap, h->d_cell_start, h->d_s_pos, h->d_s_wrap, \
        h->cap_pairs, h->d_pair_tmp, h->d_pair_key, h->d_pair_row, h->d_pair_start, h->d_pair_count, h->d_row_count, h->d_self_row, h->d_counters
        // (these kernels wait for the kernel before them on the device: their launch overlaps its tail)
        if (small_keys && rows) CU(launch_dependent(pairs_kernel<kFillSmemKeysSmall, true>, grid, kFillWarps * 32, 0, st, SOAP_PAIRS_ARGS));
        else if (small_keys) CU(launch_dependent(pairs_kernel<kFillSmemKeysSmall, false>, grid, kFillWarps * 32, 0, st, SOAP_PAIRS_ARGS));
        else if (rows) CU(launch_dependent(pairs_kernel<kFillSmemKeys, true>, grid, kFillWarps * 32, 0, st, SOAP_PAIRS_ARGS));
        else CU(launch_dependent(pairs_kernel<kFillSmemKeys, false>, grid, kFillWarps * 32, 0, st, SOAP_PAIRS_ARGS));
#undef SOAP_PAIRS_ARGS
    }
    if (!rows && !batch.struct_ptr && !brute) {
        // no Jacobian rows wanted: no row pointers, no launch order
        CU(cudaGetLastError());
        return SOAP_OK;
    }
    if (C <= kOrderMaxCenters) {
        CU(launch_dependent(rows_order_kernel, 1, 1024, 0, st, h->d_row_count, h->d_pair_count, C, row_ptr_out, h->d_order, h->d_counters));
    } else {
        scan_counts(h, h->d_row_count, row_ptr_out, C, &h->d_counters->n_rows, st);
    }
    CU(cudaGetLastError());
    return SOAP_OK;
}

int check_inputs(soap_t* h, const float* pos, const int32_t* num, int64_t N, const int32_t* centers, int64_t C,
                 const float* sites = nullptr) {
    if (!h) return SOAP_ERR_INVALID_ARG;
    if (N < 0 || C < 0 || N > 2000000000LL) return fail(h, SOAP_ERR_INVALID_ARG, "atom or centre count out of range");
    if (N > 0 && (!pos || !num)) return fail(h, SOAP_ERR_INVALID_ARG, "positions and numbers must not be NULL");
    if (!centers && !sites && C != N && C != 0) return fail(h, SOAP_ERR_INVALID_ARG, "without a centre list n_centers must equal n_atoms");
    return SOAP_OK;
}

// Plans scratch for a structure of this size: run the search (with whatever capacity there is;
// the counts come out right even when the pairs do not fit), read the totals back, grow.
int plan(soap_t* h, const float* pos, const int32_t* num, int64_t N, const Geometry& g,
         const int32_t* centers, const float* sites, int64_t C, cudaStream_t st, const Batch& batch = Batch()) {
    int rc = ensure_scratch(h, N, C, 0);
    if (rc) return rc;
    rc = launch_neighbors(h, pos, num, N, g, centers, sites, C, h->d_row_ptr, st, batch);
    if (rc) return rc;
    CU(cudaMemcpyAsync(h->h_counters, h->d_counters, sizeof(Counters), cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    const int64_t pairs = h->h_counters->n_pairs;
    h->pairs_per_center_hint = C > 0 ? (pairs + C - 1) / C : 0;
    if (pairs > h->cap_pairs) {
        rc = ensure_scratch(h, N, C, pairs + pairs / 4 + 1024);
        if (rc) return rc;
    }
    // the planning run may have reported the shortage it was there to measure: forget that bit only
    h->h_counters->status &= ~kStatusPairCapacity;
    CU(cudaMemcpyAsync(&h->d_counters->status, &h->h_counters->status, sizeof(int), cudaMemcpyHostToDevice, st));
    CU(cudaStreamSynchronize(st));
    h->planned_atoms = std::max<int64_t>(h->planned_atoms, N);
    h->planned_centers = std::max<int64_t>(h->planned_centers, C);
    return SOAP_OK;
}

void fill_center_params(soap_t* h, CenterParams& cp, const float* pos, const int32_t* centers, int64_t C,
                        const Geometry& g, bool deriv, const float* sites = nullptr) {
    cp.pos = pos; cp.centers = centers; cp.sites = sites; cp.order = C <= kOrderMaxCenters ? h->d_order : nullptr; cp.species_idx = h->d_species_idx; cp.n_centers = C; cp.geom = g;
    cp.pair_start = h->d_pair_start; cp.pair_count = h->d_pair_count; cp.pair_key = h->d_pair_key; cp.pair_row = h->d_pair_row;
    cp.row_ptr = h->d_row_ptr; cp.self_row = h->d_self_row;
    cp.pair_capacity = h->cap_pairs; cp.row_capacity = 0; cp.counters = h->d_counters;
    cp.table = h->d_table; cp.self_term = h->d_self; cp.kl = h->d_kl; cp.l_of_lm = h->d_l_of_lm;
    cp.feat_pack = h->d_feat; cp.nch_magic = (unsigned)((1ull << 32) / (unsigned)(h->n_max * (h->l_max + 1))) + 1u; cp.inv_h = h->basis.inv_h; cp.n_intervals = h->basis.n_intervals;
    cp.S = h->S; cp.n_max = h->n_max; cp.l_max = h->l_max; cp.F = (int)h->F;
    cp.P = h->P_deriv;
    cp.crossover = h->crossover; cp.emit_coeff = 0; cp.c_bar = nullptr; cp.inner_rows = 0; cp.own_scale = 1.f; cp.c_all = nullptr;
    cp.pair_w = h->weight.fn ? h->d_pair_w : nullptr; cp.w0 = (float)h->w0;
    cp.compact = 0; cp.Fc = (int)h->Fc_pitch; cp.out_center = nullptr;
    cp.out_desc = nullptr; cp.out_jac = nullptr; cp.row_atom = nullptr;
}

// Launch of the descriptor-only kernel: persistent CTAs (one per SM) whose warps take the centres in turn.
// The radial table goes to shared memory when it leaves room for at least six warps and there is enough
// work to pay for staging it; small jobs use fewer warps per CTA so that they spread over the SMs.
int launch_desc(soap_t* h, CenterParams& cp, int64_t n_work, cudaStream_t st) {
    if (n_work <= 0) return SOAP_OK;
    cp.table_ln = h->d_table_ln;
    cp.inv_h = h->basis.inv_h_values; cp.n_intervals = h->basis.n_intervals_values;      // the value table has intervals of its own
    const bool plain = center_params_plain(cp);
    const int warps_fit = (int)std::min<size_t>(kDescMaxWarps, (size_t)h->max_smem / h->desc_warp_bytes);
    // (with the table in shared memory a warp's region is a little smaller: its staged pairs are five words, not eight)
    const size_t table_pad = (h->desc_table_bytes + 15) & ~(size_t)15;
    const size_t warp_bytes_ts = (size_t)make_desc_layout(h->S, h->desc_np, h->l_max, 1, (int)(h->desc_table_bytes / 4)).per_warp * 4;
    const int warps_ts = h->desc_table_bytes > 0 && table_pad + warp_bytes_ts <= (size_t)h->max_smem
                             ? (int)std::min<size_t>(kDescMaxWarps, ((size_t)h->max_smem - table_pad) / warp_bytes_ts) : 0;
    const bool ts = plain && warps_ts >= 6 && n_work >= (int64_t)4 * h->sm_count;
    int warps = ts ? warps_ts : warps_fit;
    warps = (int)std::max<int64_t>(1, std::min<int64_t>(warps, (n_work + h->sm_count - 1) / h->sm_count));
    const unsigned grid = (unsigned)std::min<int64_t>(h->sm_count, (n_work + warps - 1) / warps);
    const size_t smem = (size_t)make_desc_layout(h->S, h->desc_np, h->l_max, warps, ts ? (int)(h->desc_table_bytes / 4) : 0).total * 4;
    CU(desc_launch(h->l_max, h->desc_np, plain, ts, cp, grid, (unsigned)warps * 32, smem, st));
    return SOAP_OK;
}

// Feature table: species pairs mu <= nu (only mu == nu without crossover), radial pair (n' >= n on
// the diagonal), l fastest.
void build_feature_table(soap_t* h) {
    h->feat_pack.clear();
    for (int mu = 0; mu < h->S; ++mu)
        for (int nu = mu; nu < (h->crossover ? h->S : mu + 1); ++nu)
            for (int n = 0; n < h->n_max; ++n)
                for (int n2 = (mu == nu ? n : 0); n2 < h->n_max; ++n2)
                    for (int l = 0; l <= h->l_max; ++l)
                        h->feat_pack.push_back(n | (n2 << 5) | (mu << 10) | (nu << 14) | (l << 18));
    h->F = (int64_t)h->feat_pack.size();
    // columns of a species-compact row: the features whose species pair involves z, in feature order
    h->compact_map.clear();
    for (int z = 0; z < h->S; ++z)
        for (int64_t f = 0; f < h->F; ++f) {
            const int pk = h->feat_pack[f];
            if (((pk >> 10) & 15) == z || ((pk >> 14) & 15) == z) h->compact_map.push_back((int)f);
        }
    h->Fc = (int64_t)h->compact_map.size() / h->S;       // the same for every species
    h->Fc_pitch = (h->Fc + 7) & ~(int64_t)7;
}

// Everything before the per-centre kernel: argument checks, device set-up, planning when the sizes
// changed, the neighbour search.
int prepare(soap_t* h, const float* pos, const int32_t* num, int64_t N, const double* cell, const int32_t* centers,
            int64_t C, long long* row_ptr_out, Geometry& g, cudaStream_t st, const float* sites = nullptr,
            const Batch& batch = Batch(), bool rows = true) {
    int rc = check_inputs(h, pos, num, N, centers, C, sites);
    if (rc) return rc;
    if (batch.struct_ptr && (h->pbc[0] || h->pbc[1] || h->pbc[2]))
        return fail(h, SOAP_ERR_INVALID_ARG, "batches of structures are for non-periodic structures");
    if ((rc = ensure_device(h))) return rc;
    if ((rc = make_geometry(h, cell, g))) return rc;
    if (h->profiling) CU(cudaEventRecord(h->ev[0], st));
    // plan (search once, read the totals, grow the scratch: allocates and waits) when this structure is larger
    // than anything planned so far; smaller ones run in the scratch that is there, and if one of them turns out
    // to have more pairs than that holds the status word says so
    if (h->planned_atoms < 0 || N > h->planned_atoms || C > h->planned_centers) {
        if ((rc = plan(h, pos, num, N, g, centers, sites, C, st, batch))) return rc;
    }
    if ((rc = launch_neighbors(h, pos, num, N, g, centers, sites, C, row_ptr_out ? row_ptr_out : h->d_row_ptr, st, batch, rows))) return rc;
    h->list_sorted = rows;
    if (h->weight.fn && C > 0) {
        pair_weight_kernel<<<(unsigned)((C + 7) / 8), 256, 0, st>>>(pos, centers, sites, C, g, h->d_pair_start, h->d_pair_count, h->d_pair_key,
                                                                   h->cap_pairs, h->d_counters, h->weight, h->d_pair_w);
        CU(cudaGetLastError());
    }
    if (h->profiling) CU(cudaEventRecord(h->ev[1], st));
    h->last_centers = C;
    return SOAP_OK;
}

int ensure_work(soap_t* h, size_t bytes) {
    if (bytes <= h->cap_work) return SOAP_OK;
    if (h->d_work) { cudaFree(h->d_work); h->d_work = nullptr; h->cap_work = 0; }
    const size_t want = bytes + bytes / 16 + 4096;
    if (cudaMalloc(&h->d_work, want) != cudaSuccess) {
        cudaGetLastError();
        return fail(h, SOAP_ERR_ALLOC, "the workspace of the averaged mode (" + std::to_string(want >> 20) +
                                           " MiB: every Jacobian row of every centre) does not fit the device; use fewer centres per call");
    }
    h->cap_work = want;
    return SOAP_OK;
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// out[col] = mean over the rows of in[rows][width], summed in a fixed order
int column_mean(soap_t* h, const float* in, int64_t rows, int width, double* partial, float* out, cudaStream_t st) {
    int chunks = (int)std::max<int64_t>(1, std::min<int64_t>(kMeanMaxChunks, rows / 32));
    const long long chunk_rows = (rows + chunks - 1) / chunks;
    chunks = (int)((rows + chunk_rows - 1) / chunk_rows);
    const unsigned gx = (unsigned)((width + kMeanThreads - 1) / kMeanThreads);
    column_partial_kernel<<<dim3(gx, (unsigned)chunks), kMeanThreads, 0, st>>>(in, rows, width, chunk_rows, partial);
    column_finish_kernel<<<gx, kMeanThreads, 0, st>>>(partial, chunks, width, 1.0 / (double)rows, out);
    CU(cudaGetLastError());
    return SOAP_OK;
}

}  // namespace

extern "C" {

int soap_create(soap_t** out, const int32_t* species, int n_species, double r_cut, int n_max, int l_max,
                double sigma, int rbf, const int pbc[3]) {
    if (!out) return SOAP_ERR_INVALID_ARG;
    *out = nullptr;
    soap_t* h = new (std::nothrow) soap_t();
    if (!h) return SOAP_ERR_ALLOC;
    auto bail = [&](int code, const std::string& msg) {
        // keep the object so that soap_last_error can be read; the caller destroys it
        h->error = msg;
        *out = h;
        return code;
    };
    if (!species || n_species < 1 || n_species > kMaxSpecies) return bail(SOAP_ERR_INVALID_ARG, "need 1 to 8 species");
    h->species.assign(species, species + n_species);
    std::sort(h->species.begin(), h->species.end());
    for (int s = 0; s < n_species; ++s) {
        if (h->species[s] < 1 || h->species[s] > 118) return bail(SOAP_ERR_INVALID_ARG, "atomic numbers must lie in 1..118");
        if (s > 0 && h->species[s] == h->species[s - 1]) return bail(SOAP_ERR_INVALID_ARG, "duplicate species");
    }
    h->S = n_species; h->n_max = n_max; h->l_max = l_max; h->rbf = rbf; h->r_cut = r_cut; h->sigma = sigma;
    for (int a = 0; a < 3; ++a) h->pbc[a] = (pbc && pbc[a]) ? 1 : 0;
    std::string err;
    int rc = build_basis(rbf, r_cut, n_max, l_max, sigma, h->basis, err);
    if (rc) return bail(rc, err);
    if ((int64_t)n_max * (l_max + 1) * (l_max + 1) > (int64_t)kMaxElemPerThread * kThreads)
        return bail(SOAP_ERR_INVALID_ARG, "n_max (l_max+1)^2 must not exceed 2048");
    build_feature_table(h);
    *out = h;
    return SOAP_OK;
}

void soap_destroy(soap_t* h) {
    if (!h) return;
    void* ptrs[] = {h->d_table, h->d_table_ln, h->d_self, h->d_kl, h->d_feat, h->d_zlut, h->d_l_of_lm, h->d_counters, h->d_bbox,
                    h->d_grid, h->d_species_idx, h->d_atom_cell, h->d_atom_wrap, h->d_s_wrap, h->d_s_pos, h->d_cell_count,
                    h->d_cell_start, h->d_pair_count, h->d_row_count, h->d_self_row, h->d_order, h->d_pair_ptr, h->d_pair_start, h->d_row_ptr, h->d_tile_sums, h->d_tile_offsets,
                    h->d_pair_key, h->d_pair_tmp, h->d_pair_row, h->d_work, h->d_pair_w, h->d_compact_map,
                    h->d_cell_tile_sums, h->d_cell_tile_offsets};
    for (void* p : ptrs) if (p) cudaFree(p);
    if (h->h_counters) cudaFreeHost(h->h_counters);
    for (cudaEvent_t e : h->ev) if (e) cudaEventDestroy(e);
    delete h;
}

int soap_num_features(const soap_t* h, int64_t* n_features) {
    if (!h || !n_features) return SOAP_ERR_INVALID_ARG;
    *n_features = h->F;
    return SOAP_OK;
}

int soap_feature_info(const soap_t* h, int64_t f, int* mu, int* nu, int* n, int* n2, int* l) {
    if (!h || f < 0 || f >= h->F) return SOAP_ERR_INVALID_ARG;
    const int pk = h->feat_pack[f];
    if (n) *n = pk & 31;
    if (n2) *n2 = (pk >> 5) & 31;
    if (mu) *mu = (pk >> 10) & 15;
    if (nu) *nu = (pk >> 14) & 15;
    if (l) *l = (pk >> 18) & 15;
    return SOAP_OK;
}

const char* soap_last_error(const soap_t* h) { return h ? h->error.c_str() : "null handle"; }

int soap_radial_table(const soap_t* h, double d, double* G, double* Ghat) {
    if (!h || !G || !Ghat || !(d >= 0) || d > h->r_cut) return SOAP_ERR_INVALID_ARG;
    eval_table(h->basis, d, G, Ghat);
    return SOAP_OK;
}

static int neighbors_impl(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms, const double* cell,
                          const int32_t* d_centers, const float* d_sites, int64_t n_centers, int64_t* n_pairs, int64_t* n_rows,
                          void* stream, const Batch& batch = Batch()) {
    int rc = check_inputs(h, d_positions, d_numbers, n_atoms, d_centers, n_centers, d_sites);
    if (rc) return rc;
    if (batch.struct_ptr && (h->pbc[0] || h->pbc[1] || h->pbc[2]))
        return fail(h, SOAP_ERR_INVALID_ARG, "batches of structures are for non-periodic structures");
    if ((rc = ensure_device(h))) return rc;
    Geometry g;
    if ((rc = make_geometry(h, cell, g))) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if ((rc = plan(h, d_positions, d_numbers, n_atoms, g, d_centers, d_sites, n_centers, st, batch))) return rc;
    if ((rc = launch_neighbors(h, d_positions, d_numbers, n_atoms, g, d_centers, d_sites, n_centers, h->d_row_ptr, st, batch))) return rc;
    h->list_sorted = true;
    CU(cudaMemcpyAsync(h->h_counters, h->d_counters, sizeof(Counters), cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    h->last_centers = n_centers;
    if (n_pairs) *n_pairs = h->h_counters->n_pairs;
    if (n_rows) *n_rows = h->h_counters->n_rows;
    return SOAP_OK;
}

int soap_neighbors(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms, const double* cell,
                   const int32_t* d_centers, int64_t n_centers, int64_t* n_pairs, int64_t* n_rows, void* stream) {
    return neighbors_impl(h, d_positions, d_numbers, n_atoms, cell, d_centers, nullptr, n_centers, n_pairs, n_rows, stream);
}

int soap_neighbors_at(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms, const double* cell,
                      const float* d_sites, int64_t n_sites, int64_t* n_pairs, int64_t* n_rows, void* stream) {
    if (h && n_sites > 0 && !d_sites) return fail(h, SOAP_ERR_INVALID_ARG, "d_sites must not be NULL");
    static const float none[3] = {0.f, 0.f, 0.f};
    return neighbors_impl(h, d_positions, d_numbers, n_atoms, cell, nullptr, d_sites ? d_sites : none, n_sites, n_pairs, n_rows, stream);
}

int soap_neighbor_list(soap_t* h, int64_t* d_pair_ptr, int32_t* d_pair_atom, int32_t* d_pair_shift,
                       int64_t capacity_pairs, void* stream) {
    if (!h || !d_pair_ptr || !d_pair_atom || capacity_pairs < 0) return SOAP_ERR_INVALID_ARG;
    if (!h->tables_ready || h->planned_atoms < 0) return fail(h, SOAP_ERR_INVALID_ARG, "no neighbour list has been built yet");
    if (!h->list_sorted) return fail(h, SOAP_ERR_INVALID_ARG, "the last call was descriptor-only and kept its pairs unsorted: call soap_neighbors first");
    cudaStream_t st = (cudaStream_t)stream;
    // the pair arrays are addressed by segment: make the compact row pointers first, then gather
    scan_counts(h, h->d_pair_count, (long long*)d_pair_ptr, h->last_centers, nullptr, st);
    export_pairs_kernel<<<256, 256, 0, st>>>(h->d_pair_start, (const long long*)d_pair_ptr, h->d_pair_key, h->last_centers,
                                             capacity_pairs, d_pair_atom, d_pair_shift, h->d_counters);
    CU(cudaGetLastError());
    return SOAP_OK;
}

static int descriptor_impl(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms, const double* cell,
                           const int32_t* d_centers, const float* d_sites, int64_t n_centers, float* d_out, void* stream,
                           const Batch& batch = Batch()) {
    if (h && n_centers > 0 && !d_out) return fail(h, SOAP_ERR_INVALID_ARG, "d_out must not be NULL");
    Geometry g;
    cudaStream_t st = (cudaStream_t)stream;
    int rc = prepare(h, d_positions, d_numbers, n_atoms, cell, d_centers, n_centers, nullptr, g, st, d_sites, batch, false);
    if (rc) return rc;
    if (n_centers > 0) {
        CenterParams cp;
        fill_center_params(h, cp, d_positions, d_centers, n_centers, g, false, d_sites);
        cp.out_desc = d_out;
        if ((rc = launch_desc(h, cp, n_centers, st))) return rc;
    }
    if (h->profiling) CU(cudaEventRecord(h->ev[2], st));
    return SOAP_OK;
}

int soap_descriptor(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms, const double* cell,
                    const int32_t* d_centers, int64_t n_centers, float* d_out, void* stream) {
    return descriptor_impl(h, d_positions, d_numbers, n_atoms, cell, d_centers, nullptr, n_centers, d_out, stream);
}

int soap_descriptor_at(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms, const double* cell,
                       const float* d_sites, int64_t n_sites, float* d_out, void* stream) {
    if (h && !d_sites) return n_sites == 0 ? SOAP_OK : fail(h, SOAP_ERR_INVALID_ARG, "d_sites must not be NULL");
    return descriptor_impl(h, d_positions, d_numbers, n_atoms, cell, nullptr, d_sites, n_sites, d_out, stream);
}

static int derivatives_impl(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms, const double* cell,
                            const int32_t* d_centers, const float* d_sites, int64_t n_centers, float* d_out_desc, float* d_out_jac,
                            int64_t capacity_rows, int64_t* d_row_ptr, int32_t* d_row_atom, void* stream,
                            float* d_out_center = nullptr, const Batch& batch = Batch()) {
    if (h && (!d_row_ptr || capacity_rows < 0)) return fail(h, SOAP_ERR_INVALID_ARG, "d_row_ptr must not be NULL");
    if (h && n_centers > 0 && (!d_out_desc || !d_out_jac || !d_row_atom)) return fail(h, SOAP_ERR_INVALID_ARG, "output pointers must not be NULL");
    Geometry g;
    cudaStream_t st = (cudaStream_t)stream;
    int rc = prepare(h, d_positions, d_numbers, n_atoms, cell, d_centers, n_centers, (long long*)d_row_ptr, g, st, d_sites, batch);
    if (rc) return rc;
    if (n_centers > 0) {
        CenterParams cp;
        fill_center_params(h, cp, d_positions, d_centers, n_centers, g, true, d_sites);
        cp.row_ptr = (const long long*)d_row_ptr;
        cp.row_capacity = capacity_rows;
        cp.out_desc = d_out_desc; cp.out_jac = d_out_jac; cp.row_atom = d_row_atom;
        if (d_out_center) { cp.compact = 1; cp.out_center = d_out_center; }
        CU(center_launch(kCenterDeriv, h->l_max, h->n_max, cp, (unsigned)n_centers, h->smem_deriv, st));
    }
    if (h->profiling) CU(cudaEventRecord(h->ev[2], st));
    return SOAP_OK;
}

int soap_derivatives(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms, const double* cell,
                     const int32_t* d_centers, int64_t n_centers, float* d_out_desc, float* d_out_jac,
                     int64_t capacity_rows, int64_t* d_row_ptr, int32_t* d_row_atom, void* stream) {
    return derivatives_impl(h, d_positions, d_numbers, n_atoms, cell, d_centers, nullptr, n_centers, d_out_desc, d_out_jac,
                            capacity_rows, d_row_ptr, d_row_atom, stream);
}

int soap_derivatives_at(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms, const double* cell,
                        const float* d_sites, int64_t n_sites, float* d_out_desc, float* d_out_jac,
                        int64_t capacity_rows, int64_t* d_row_ptr, int32_t* d_row_atom, void* stream) {
    if (h && !d_sites && n_sites > 0) return fail(h, SOAP_ERR_INVALID_ARG, "d_sites must not be NULL");
    static const float none[3] = {0.f, 0.f, 0.f};
    return derivatives_impl(h, d_positions, d_numbers, n_atoms, cell, nullptr, d_sites ? d_sites : none, n_sites, d_out_desc,
                            d_out_jac, capacity_rows, d_row_ptr, d_row_atom, stream);
}

// ---- many independent structures in one call ----
static int check_batch(soap_t* h, const int64_t* d_struct_ptr, int64_t n_structs, int64_t n_atoms) {
    if (!h) return SOAP_ERR_INVALID_ARG;
    if (n_structs < 0 || (n_atoms > 0 && n_structs < 1)) return fail(h, SOAP_ERR_INVALID_ARG, "n_structs must be at least 1 when there are atoms");
    if (n_structs > 0 && !d_struct_ptr) return fail(h, SOAP_ERR_INVALID_ARG, "d_struct_ptr must not be NULL");
    return SOAP_OK;
}

int soap_neighbors_batch(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms,
                         const int64_t* d_struct_ptr, int64_t n_structs, int64_t* n_pairs, int64_t* n_rows, void* stream) {
    int rc = check_batch(h, d_struct_ptr, n_structs, n_atoms);
    if (rc) return rc;
    static const long long none[2] = {0, 0};
    Batch b;
    b.struct_ptr = d_struct_ptr ? (const long long*)d_struct_ptr : none;
    b.n_structs = n_structs;
    return neighbors_impl(h, d_positions, d_numbers, n_atoms, nullptr, nullptr, nullptr, n_atoms, n_pairs, n_rows, stream, b);
}

int soap_descriptor_batch(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms,
                          const int64_t* d_struct_ptr, int64_t n_structs, float* d_out, void* stream) {
    int rc = check_batch(h, d_struct_ptr, n_structs, n_atoms);
    if (rc) return rc;
    static const long long none[2] = {0, 0};
    Batch b;
    b.struct_ptr = d_struct_ptr ? (const long long*)d_struct_ptr : none;
    b.n_structs = n_structs;
    return descriptor_impl(h, d_positions, d_numbers, n_atoms, nullptr, nullptr, nullptr, n_atoms, d_out, stream, b);
}

int soap_derivatives_batch(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms,
                           const int64_t* d_struct_ptr, int64_t n_structs, float* d_out_desc, float* d_out_jac,
                           int64_t capacity_rows, int64_t* d_row_ptr, int32_t* d_row_atom, void* stream) {
    int rc = check_batch(h, d_struct_ptr, n_structs, n_atoms);
    if (rc) return rc;
    static const long long none[2] = {0, 0};
    Batch b;
    b.struct_ptr = d_struct_ptr ? (const long long*)d_struct_ptr : none;
    b.n_structs = n_structs;
    return derivatives_impl(h, d_positions, d_numbers, n_atoms, nullptr, nullptr, nullptr, n_atoms, d_out_desc, d_out_jac,
                            capacity_rows, d_row_ptr, d_row_atom, stream, nullptr, b);
}

int soap_num_compact_features(const soap_t* h, int64_t* n_compact, int64_t* pitch) {
    if (!h) return SOAP_ERR_INVALID_ARG;
    if (n_compact) *n_compact = h->Fc;
    if (pitch) *pitch = h->Fc_pitch;
    return SOAP_OK;
}

int soap_compact_feature_map(const soap_t* h, int species_index, int32_t* map) {
    if (!h || !map || species_index < 0 || species_index >= h->S) return SOAP_ERR_INVALID_ARG;
    std::memcpy(map, h->compact_map.data() + (size_t)species_index * h->Fc, (size_t)h->Fc * sizeof(int32_t));
    return SOAP_OK;
}

int soap_derivatives_compact(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms, const double* cell,
                             const int32_t* d_centers, int64_t n_centers, float* d_out_desc, float* d_out_center,
                             float* d_out_jac, int64_t capacity_rows, int64_t* d_row_ptr, int32_t* d_row_atom, void* stream) {
    if (h && n_centers > 0 && !d_out_center) return fail(h, SOAP_ERR_INVALID_ARG, "d_out_center must not be NULL");
    return derivatives_impl(h, d_positions, d_numbers, n_atoms, cell, d_centers, nullptr, n_centers, d_out_desc, d_out_jac,
                            capacity_rows, d_row_ptr, d_row_atom, stream, n_centers > 0 ? d_out_center : nullptr);
}

int soap_compact_expand(soap_t* h, const int32_t* d_numbers, const int32_t* d_centers, int64_t n_centers,
                        const float* d_center_rows, const float* d_jac_compact, const int64_t* d_row_ptr,
                        const int32_t* d_row_atom, float* d_out_rows, void* stream) {
    if (!h) return SOAP_ERR_INVALID_ARG;
    if (n_centers < 0) return fail(h, SOAP_ERR_INVALID_ARG, "negative size");
    if (n_centers == 0) return SOAP_OK;
    if (!d_numbers || !d_center_rows || !d_jac_compact || !d_row_ptr || !d_row_atom || !d_out_rows) return fail(h, SOAP_ERR_INVALID_ARG, "NULL pointer");
    int rc = ensure_device(h);
    if (rc) return rc;
    if (!h->d_compact_map) CU(upload(&h->d_compact_map, h->compact_map));
    compact_expand_kernel<<<(unsigned)n_centers, 256, 0, (cudaStream_t)stream>>>(
        d_jac_compact, d_center_rows, (const long long*)d_row_ptr, d_row_atom, d_centers, d_numbers, h->d_zlut,
        h->d_compact_map, (int)h->Fc, (int)h->Fc_pitch, (int)h->F, d_out_rows);
    CU(cudaGetLastError());
    return SOAP_OK;
}

int soap_rows_dense(soap_t* h, const float* d_rows, int64_t width, const int64_t* d_row_ptr, const int32_t* d_row_atom,
                    int64_t n_centers, const int32_t* d_include, int64_t n_include, float* d_out, void* stream) {
    if (!h) return SOAP_ERR_INVALID_ARG;
    if (n_centers < 0 || n_include < 0 || width < 1 || width > 2147483647LL / 3) return fail(h, SOAP_ERR_INVALID_ARG, "size out of range");
    if (n_centers == 0 || n_include == 0) return SOAP_OK;
    if (!d_rows || !d_row_ptr || !d_row_atom || !d_out) return fail(h, SOAP_ERR_INVALID_ARG, "NULL pointer");
    if (n_centers * n_include > 2147483647LL) return fail(h, SOAP_ERR_INVALID_ARG, "more than 2^31-1 (centre, atom) slots: split the call");
    dense_scatter_kernel<<<(unsigned)(n_centers * n_include), 128, 0, (cudaStream_t)stream>>>(
        d_rows, (const long long*)d_row_ptr, d_row_atom, n_centers, d_include, n_include, (int)width, d_out);
    CU(cudaGetLastError());
    return SOAP_OK;
}

int soap_jacobian_dense(soap_t* h, const float* d_jac_rows, const int64_t* d_row_ptr, const int32_t* d_row_atom,
                        int64_t n_centers, const int32_t* d_include, int64_t n_include, float* d_out, void* stream) {
    if (!h) return SOAP_ERR_INVALID_ARG;
    return soap_rows_dense(h, d_jac_rows, h->F, d_row_ptr, d_row_atom, n_centers, d_include, n_include, d_out, stream);
}

int soap_set_crossover(soap_t* h, int crossover) {
    if (!h) return SOAP_ERR_INVALID_ARG;
    crossover = crossover ? 1 : 0;
    if (crossover == h->crossover) return SOAP_OK;
    h->crossover = crossover;
    build_feature_table(h);
    if (h->tables_ready) {
        CU(cudaDeviceSynchronize());
        cudaFree(h->d_feat);
        h->d_feat = nullptr;
        CU(upload(&h->d_feat, h->feat_pack));
        if (h->d_compact_map) { cudaFree(h->d_compact_map); h->d_compact_map = nullptr; }
    }
    return SOAP_OK;
}

int soap_set_weighting(soap_t* h, int function, double r0, double c, double d, double m, double w0) {
    if (!h) return SOAP_ERR_INVALID_ARG;
    if (function < SOAP_WEIGHT_NONE || function > SOAP_WEIGHT_EXP) return fail(h, SOAP_ERR_INVALID_ARG, "unknown weighting function");
    if (function != SOAP_WEIGHT_NONE) {
        if (!(r0 > 0) || !std::isfinite(c) || !std::isfinite(w0)) return fail(h, SOAP_ERR_INVALID_ARG, "weighting needs r0 > 0 and finite c, w0");
        if (function == SOAP_WEIGHT_POLY && !(m >= 0)) return fail(h, SOAP_ERR_INVALID_ARG, "poly weighting needs m >= 0");
        if (function == SOAP_WEIGHT_POW && (!(m >= 0) || !(d > 0))) return fail(h, SOAP_ERR_INVALID_ARG, "pow weighting needs m >= 0 and d > 0");
        if (function == SOAP_WEIGHT_EXP && !(d >= 0)) return fail(h, SOAP_ERR_INVALID_ARG, "exp weighting needs d >= 0");
    }
    const bool was = h->weight.fn != 0, now = function != SOAP_WEIGHT_NONE;
    h->weight = WeightParams{function, now ? r0 : 1.0, now ? c : 1.0, d, m};
    h->w0 = now ? w0 : 1.0;
    if (was != now) {
        // the pair scratch gains or loses the weight array and the kernels' shared memory changes
        h->planned_atoms = -1;
        if (h->tables_ready) {
            CU(cudaDeviceSynchronize());
            if (h->d_pair_w) { cudaFree(h->d_pair_w); h->d_pair_w = nullptr; }
            if (now) CU(regrow(&h->d_pair_w, (size_t)std::max<int64_t>(h->cap_pairs, 1)));
            if (int rc = plan_smem(h)) return rc;
        }
    }
    return SOAP_OK;
}

int soap_num_coefficients(const soap_t* h, int64_t* n_coefficients) {
    if (!h || !n_coefficients) return SOAP_ERR_INVALID_ARG;
    *n_coefficients = (int64_t)h->S * h->n_max * (h->l_max + 1) * (h->l_max + 1);
    return SOAP_OK;
}

int soap_coefficients(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms, const double* cell,
                      const int32_t* d_centers, int64_t n_centers, float* d_out, void* stream) {
    if (h && n_centers > 0 && !d_out) return fail(h, SOAP_ERR_INVALID_ARG, "d_out must not be NULL");
    Geometry g;
    cudaStream_t st = (cudaStream_t)stream;
    int rc = prepare(h, d_positions, d_numbers, n_atoms, cell, d_centers, n_centers, nullptr, g, st, nullptr, Batch(), false);
    if (rc) return rc;
    if (n_centers > 0) {
        CenterParams cp;
        fill_center_params(h, cp, d_positions, d_centers, n_centers, g, false);
        cp.out_desc = d_out;
        cp.emit_coeff = 1;
        if ((rc = launch_desc(h, cp, n_centers, st))) return rc;
    }
    if (h->profiling) CU(cudaEventRecord(h->ev[2], st));
    return SOAP_OK;
}

int soap_coefficient_derivatives(soap_t* h, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms,
                                 const double* cell, const int32_t* d_centers, int64_t n_centers, float* d_out_coeff,
                                 float* d_out_jac, int64_t capacity_rows, int64_t* d_row_ptr, int32_t* d_row_atom,
                                 void* stream) {
    if (h && (!d_row_ptr || capacity_rows < 0)) return fail(h, SOAP_ERR_INVALID_ARG, "d_row_ptr must not be NULL");
    if (h && n_centers > 0 && (!d_out_coeff || !d_out_jac || !d_row_atom)) return fail(h, SOAP_ERR_INVALID_ARG, "output pointers must not be NULL");
    Geometry g;
    cudaStream_t st = (cudaStream_t)stream;
    int rc = prepare(h, d_positions, d_numbers, n_atoms, cell, d_centers, n_centers, (long long*)d_row_ptr, g, st);
    if (rc) return rc;
    if (n_centers > 0) {
        CenterParams cp;
        fill_center_params(h, cp, d_positions, d_centers, n_centers, g, true);
        cp.row_ptr = (const long long*)d_row_ptr;
        cp.row_capacity = capacity_rows;
        cp.out_desc = d_out_coeff; cp.out_jac = d_out_jac; cp.row_atom = d_row_atom;
        CU(center_launch(kCenterCoeff, h->l_max, h->n_max, cp, (unsigned)n_centers, h->smem_deriv, st));
    }
    if (h->profiling) CU(cudaEventRecord(h->ev[2], st));
    return SOAP_OK;
}

int soap_descriptor_average(soap_t* h, int mode, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms,
                            const double* cell, const int32_t* d_centers, int64_t n_centers, float* d_out, void* stream) {
    if (!h) return SOAP_ERR_INVALID_ARG;
    if (mode != SOAP_AVERAGE_INNER && mode != SOAP_AVERAGE_OUTER) return fail(h, SOAP_ERR_INVALID_ARG, "mode must be SOAP_AVERAGE_INNER or SOAP_AVERAGE_OUTER");
    if (n_centers < 1) return fail(h, SOAP_ERR_INVALID_ARG, "an average needs at least one centre");
    if (!d_out) return fail(h, SOAP_ERR_INVALID_ARG, "d_out must not be NULL");
    Geometry g;
    cudaStream_t st = (cudaStream_t)stream;
    int rc = prepare(h, d_positions, d_numbers, n_atoms, cell, d_centers, n_centers, nullptr, g, st, nullptr, Batch(), false);
    if (rc) return rc;
    const int F = (int)h->F, W = h->S * h->n_max * (h->l_max + 1) * (h->l_max + 1);
    const bool inner = mode == SOAP_AVERAGE_INNER;
    const int width = inner ? W : F;
    const size_t o_rows = 0, o_partial = align256((size_t)n_centers * width * 4),
                 o_cbar = o_partial + align256((size_t)kMeanMaxChunks * width * 8), total = o_cbar + align256((size_t)W * 4);
    if ((rc = ensure_work(h, total))) return rc;
    char* w = (char*)h->d_work;
    CenterParams cp;
    fill_center_params(h, cp, d_positions, d_centers, n_centers, g, false);
    cp.out_desc = (float*)(w + o_rows);
    cp.emit_coeff = inner ? 1 : 0;
    if ((rc = launch_desc(h, cp, n_centers, st))) return rc;
    if ((rc = column_mean(h, (const float*)(w + o_rows), n_centers, width, (double*)(w + o_partial),
                          inner ? (float*)(w + o_cbar) : d_out, st))) return rc;
    if (inner) {
        // Eq. 4 on the mean coefficients: one CTA, no pairs
        cp.emit_coeff = 0;
        cp.c_bar = (const float*)(w + o_cbar);
        cp.out_desc = d_out;
        cp.order = nullptr;
        if ((rc = launch_desc(h, cp, 1, st))) return rc;
    }
    if (h->profiling) CU(cudaEventRecord(h->ev[2], st));
    return SOAP_OK;
}

int soap_derivatives_average(soap_t* h, int mode, const float* d_positions, const int32_t* d_numbers, int64_t n_atoms,
                             const double* cell, const int32_t* d_centers, int64_t n_centers, float* d_out_desc,
                             float* d_out_jac, void* stream) {
    if (!h) return SOAP_ERR_INVALID_ARG;
    if (mode != SOAP_AVERAGE_INNER && mode != SOAP_AVERAGE_OUTER) return fail(h, SOAP_ERR_INVALID_ARG, "mode must be SOAP_AVERAGE_INNER or SOAP_AVERAGE_OUTER");
    if (n_centers < 1) return fail(h, SOAP_ERR_INVALID_ARG, "an average needs at least one centre");
    if (!d_out_desc || !d_out_jac) return fail(h, SOAP_ERR_INVALID_ARG, "output pointers must not be NULL");
    Geometry g;
    cudaStream_t st = (cudaStream_t)stream;
    int rc = prepare(h, d_positions, d_numbers, n_atoms, cell, d_centers, n_centers, nullptr, g, st);
    if (rc) return rc;
    if (mode == SOAP_AVERAGE_INNER && !d_centers && n_centers == n_atoms) {
        // Inner average with every atom a centre: pbar = P(cbar) and d pbar / d r_a = dP/dcbar . (1/C) sum_i grad_a c(i).
        // Centre i sees atom a where a sees i, mirrored, so the kernel of atom a collects that sum from its own
        // pairs in pass 1 and contracts it with cbar like a centre's own row: no per-pair rows, no workspace for them.
        const int W = h->S * h->n_max * (h->l_max + 1) * (h->l_max + 1);
        const size_t o_rows = 0, o_partial = align256((size_t)n_centers * W * 4),
                     o_cbar = o_partial + align256((size_t)kMeanMaxChunks * W * 8), total = o_cbar + align256((size_t)W * 4);
        if ((rc = ensure_work(h, total))) return rc;
        char* w = (char*)h->d_work;
        CenterParams cp;
        fill_center_params(h, cp, d_positions, d_centers, n_centers, g, false);
        cp.out_desc = (float*)(w + o_rows);
        cp.emit_coeff = 1;
        if ((rc = launch_desc(h, cp, n_centers, st))) return rc;
        if ((rc = column_mean(h, (const float*)(w + o_rows), n_centers, W, (double*)(w + o_partial), (float*)(w + o_cbar), st))) return rc;
        fill_center_params(h, cp, d_positions, d_centers, n_centers, g, true);
        cp.row_capacity = INT64_MAX;
        cp.c_bar = (const float*)(w + o_cbar);
        cp.out_desc = d_out_desc;
        cp.out_jac = d_out_jac;
        cp.inner_rows = 1;
        cp.own_scale = (float)(1.0 / (double)n_centers);
        CU(center_launch(kCenterInner, h->l_max, h->n_max, cp, (unsigned)n_centers, h->smem_deriv, st));
        if (h->profiling) CU(cudaEventRecord(h->ev[2], st));
        return SOAP_OK;
    }
    if (mode == SOAP_AVERAGE_OUTER && !d_centers && n_centers == n_atoms && h->outer_fast) {
        // Outer average with every atom a centre: atom a gathers its own row and the rows that the centres it sees
        // hold for it (they need those centres' coefficients, written first by the descriptor kernel): one row per
        // atom, no per-pair rows, no workspace for them.
        const int F = (int)h->F, W = h->S * h->n_max * (h->l_max + 1) * (h->l_max + 1);
        const size_t o_coeff = 0, o_rows = align256((size_t)n_centers * W * 4),
                     o_partial = o_rows + align256((size_t)n_centers * F * 4), total = o_partial + align256((size_t)kMeanMaxChunks * F * 8);
        if ((rc = ensure_work(h, total))) return rc;
        char* w = (char*)h->d_work;
        CenterParams cp;
        fill_center_params(h, cp, d_positions, d_centers, n_centers, g, false);
        cp.out_desc = (float*)(w + o_coeff);
        cp.emit_coeff = 1;
        if ((rc = launch_desc(h, cp, n_centers, st))) return rc;
        fill_center_params(h, cp, d_positions, d_centers, n_centers, g, true);
        cp.row_capacity = INT64_MAX;
        cp.c_all = (const float*)(w + o_coeff);
        cp.out_desc = (float*)(w + o_rows);
        cp.out_jac = d_out_jac;
        cp.own_scale = (float)(1.0 / (double)n_centers);
        cp.P = h->P_outer;
        CU(center_launch(kCenterOuter, h->l_max, h->n_max, cp, (unsigned)n_centers, h->smem_outer, st));
        if ((rc = column_mean(h, (const float*)(w + o_rows), n_centers, F, (double*)(w + o_partial), d_out_desc, st))) return rc;
        if (h->profiling) CU(cudaEventRecord(h->ev[2], st));
        return SOAP_OK;
    }
    // the row total sizes the workspace; a structure that outgrew its plan is planned again
    CU(cudaMemcpyAsync(h->h_counters, h->d_counters, sizeof(Counters), cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    if (h->h_counters->n_pairs > h->cap_pairs) {
        h->planned_atoms = -1;
        if ((rc = prepare(h, d_positions, d_numbers, n_atoms, cell, d_centers, n_centers, nullptr, g, st))) return rc;
        CU(cudaMemcpyAsync(h->h_counters, h->d_counters, sizeof(Counters), cudaMemcpyDeviceToHost, st));
        CU(cudaStreamSynchronize(st));
    }
    const int64_t rows = h->h_counters->n_rows;
    const int F = (int)h->F, W = h->S * h->n_max * (h->l_max + 1) * (h->l_max + 1);
    const bool inner = mode == SOAP_AVERAGE_INNER;
    const int width = inner ? W : F;
    const size_t o_jac = 0, o_atom = align256((size_t)rows * 3 * F * 4), o_rows = o_atom + align256((size_t)rows * 4),
                 o_partial = o_rows + align256((size_t)n_centers * width * 4),
                 o_cbar = o_partial + align256((size_t)kMeanMaxChunks * width * 8), total = o_cbar + align256((size_t)W * 4);
    if ((rc = ensure_work(h, total))) return rc;
    char* w = (char*)h->d_work;
    CenterParams cp;
    if (inner) {
        fill_center_params(h, cp, d_positions, d_centers, n_centers, g, false);
        cp.out_desc = (float*)(w + o_rows);
        cp.emit_coeff = 1;
        if ((rc = launch_desc(h, cp, n_centers, st))) return rc;
        if ((rc = column_mean(h, (const float*)(w + o_rows), n_centers, W, (double*)(w + o_partial), (float*)(w + o_cbar), st))) return rc;
    }
    fill_center_params(h, cp, d_positions, d_centers, n_centers, g, true);
    cp.row_capacity = rows;
    cp.out_jac = (float*)(w + o_jac);
    cp.row_atom = (int*)(w + o_atom);
    if (inner) {
        // every centre differentiates against the mean coefficients; the first one writes the descriptor
        cp.c_bar = (const float*)(w + o_cbar);
        cp.out_desc = d_out_desc;
    } else {
        cp.out_desc = (float*)(w + o_rows);
    }
    CU(center_launch(kCenterDeriv, h->l_max, h->n_max, cp, (unsigned)n_centers, h->smem_deriv, st));
    if (!inner && (rc = column_mean(h, (const float*)(w + o_rows), n_centers, F, (double*)(w + o_partial), d_out_desc, st))) return rc;
    if (n_atoms > 0) {
        const int width3 = 3 * F;
        int slices = (int)std::max<int64_t>(1, std::min<int64_t>((1184 + n_atoms - 1) / n_atoms, (width3 + kAvgThreads - 1) / kAvgThreads));
        const int slice = (((width3 + slices - 1) / slices) + 31) & ~31;
        slices = (width3 + slice - 1) / slice;
        average_rows_kernel<<<dim3((unsigned)n_atoms, (unsigned)slices), kAvgThreads, 0, st>>>(
            (const float*)(w + o_jac), h->d_row_ptr, (const int*)(w + o_atom), n_centers, width3, slice,
            (float)(1.0 / (double)n_centers), d_out_jac);
        CU(cudaGetLastError());
    }
    if (h->profiling) CU(cudaEventRecord(h->ev[2], st));
    return SOAP_OK;
}

int soap_status(soap_t* h, int64_t* n_pairs, int64_t* n_rows, void* stream) {
    if (!h) return SOAP_ERR_INVALID_ARG;
    if (!h->tables_ready) return SOAP_OK;
    cudaStream_t st = (cudaStream_t)stream;
    CU(cudaMemcpyAsync(h->h_counters, h->d_counters, sizeof(Counters), cudaMemcpyDeviceToHost, st));
    CU(cudaMemsetAsync(&h->d_counters->status, 0, sizeof(int), st));
    CU(cudaStreamSynchronize(st));
    if (n_pairs) *n_pairs = h->h_counters->n_pairs;
    if (n_rows) *n_rows = h->h_counters->n_rows;
    const int s = h->h_counters->status;
    if (s & kStatusUnknownSpecies) return fail(h, SOAP_ERR_UNKNOWN_SPECIES, "an atomic number is not in the species list");
    if (s & kStatusShiftRange) return fail(h, SOAP_ERR_INVALID_ARG, "positions lie too many cells away from the unit cell");
    if (s & kStatusPairCapacity) return fail(h, SOAP_ERR_CAPACITY, "more pairs than planned (call soap_neighbors again) or than the export buffer holds");
    if (s & kStatusRowCapacity) return fail(h, SOAP_ERR_CAPACITY, "more Jacobian rows than capacity_rows");
    return SOAP_OK;
}

// ---------------------------------------------------------------------------------------------
// Neighbour counts without any allocation.
//
// Some hosts of this library may not allocate device memory when they call it: code that runs
// inside a memory pool it must not disturb, a real-time loop where cudaMalloc's implicit
// synchronisation is not acceptable, or a process whose memory budget was handed out in full at
// start-up.  For them the cell list lives in the fixed array below, which every GPU that loads the
// library carries until the process exits.
constexpr int kStaticMaxAtoms = 65536;
constexpr int kStaticMaxCells = 65536;
struct StaticLayout {
    static constexpr size_t header = 1024;                                       // bbox, grid, counters
    static constexpr size_t atom_cell = header;
    static constexpr size_t atom_wrap = atom_cell + sizeof(int) * kStaticMaxAtoms;
    static constexpr size_t s_wrap = atom_wrap + sizeof(int) * kStaticMaxAtoms;
    static constexpr size_t s_pos = s_wrap + sizeof(int) * kStaticMaxAtoms;
    static constexpr size_t cell_count = s_pos + sizeof(float4) * kStaticMaxAtoms;
    static constexpr size_t cell_start = cell_count + 256 * ((sizeof(int) * (kStaticMaxCells + 1) + 255) / 256);
    static constexpr size_t total = cell_start + 256 * ((sizeof(int) * (kStaticMaxCells + 1) + 255) / 256);
};
static __device__ __align__(256) unsigned char g_static_scratch[StaticLayout::total];   // about 2.4 MB

// bounding box only (the handle-based path also looks up species here; this one has no species)
__global__ void bbox_only_kernel(const float* __restrict__ pos, long long N, Geometry geom, unsigned long long* bbox) {
    double hi[3] = {-1e300, -1e300, -1e300}, lo[3] = {-1e300, -1e300, -1e300};
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < N; i += (long long)gridDim.x * blockDim.x) {
        double f[3];
        frac_coords(geom, pos[3 * i], pos[3 * i + 1], pos[3 * i + 2], f);
        for (int a = 0; a < 3; ++a) { hi[a] = fmax(hi[a], f[a]); lo[a] = fmax(lo[a], -f[a]); }
    }
    for (int a = 0; a < 3; ++a)
        for (int o = 16; o > 0; o >>= 1) {
            hi[a] = fmax(hi[a], __shfl_xor_sync(0xffffffffu, hi[a], o));
            lo[a] = fmax(lo[a], __shfl_xor_sync(0xffffffffu, lo[a], o));
        }
    if ((threadIdx.x & 31) == 0)
        for (int a = 0; a < 3; ++a) {
            atomicMax(&bbox[a], enc_double(hi[a]));
            atomicMax(&bbox[3 + a], enc_double(lo[a]));
        }
}

int soap_neighbor_counts_static(const float* d_positions, int64_t n_atoms, double r_cut, int32_t* d_counts,
                                void* stream, char* message, int64_t message_len) {
    auto say = [&](int code, const char* text) {
        if (message && message_len > 0) std::snprintf(message, (size_t)message_len, "%s", text);
        return code;
    };
    if (n_atoms < 0 || !(r_cut > 0) || (n_atoms > 0 && (!d_positions || !d_counts)))
        return say(SOAP_ERR_INVALID_ARG, "need n_atoms >= 0, r_cut > 0 and non-NULL device pointers");
    if (n_atoms > kStaticMaxAtoms)
        return say(SOAP_ERR_CAPACITY, "soap_neighbor_counts_static handles at most 65536 atoms (fixed scratch); "
                                       "use soap_neighbors for larger structures");
    // Set-up, once per device: the array's name is only a host-side stand-in here, so ask the
    // runtime for its device address.  The first call on a device does this (it may initialise
    // the context) and should therefore come before any stream capture.
    static std::atomic<unsigned char*> base_of_device[64];    // zero-initialised; one look-up per device, published atomically
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return say(SOAP_ERR_CUDA, cudaGetErrorString(e));
    if (dev < 0 || dev >= 64) return say(SOAP_ERR_INVALID_ARG, "device ordinal out of range");
    unsigned char* base = base_of_device[dev].load(std::memory_order_acquire);
    if (!base) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr) return say(SOAP_ERR_CUDA, cudaGetErrorString(e));
        base = static_cast<unsigned char*>(ptr);
        base_of_device[dev].store(base, std::memory_order_release);
    }
    unsigned long long* bbox = reinterpret_cast<unsigned long long*>(base);
    GridParams* grid = reinterpret_cast<GridParams*>(base + 256);
    Counters* counters = reinterpret_cast<Counters*>(base + 768);
    int* atom_cell = reinterpret_cast<int*>(base + StaticLayout::atom_cell);
    int* atom_wrap = reinterpret_cast<int*>(base + StaticLayout::atom_wrap);
    int* s_wrap = reinterpret_cast<int*>(base + StaticLayout::s_wrap);
    float4* s_pos = reinterpret_cast<float4*>(base + StaticLayout::s_pos);
    int* cell_count = reinterpret_cast<int*>(base + StaticLayout::cell_count);
    int* cell_start = reinterpret_cast<int*>(base + StaticLayout::cell_start);
    if (n_atoms == 0) return SOAP_OK;
    Geometry g;
    const double ident[9] = {1, 0, 0, 0, 1, 0, 0, 0, 1};
    std::memcpy(g.cell, ident, sizeof(ident));
    std::memcpy(g.inv, ident, sizeof(ident));
    for (int a = 0; a < 3; ++a) { g.height[a] = 1.0; g.pbc[a] = 0; }
    g.r_cut = r_cut;
    g.rc2 = r_cut * r_cut;
    cudaStream_t st = (cudaStream_t)stream;
    const long long N = n_atoms;
    // the array keeps whatever the previous call left: clear what has to start at zero
    if ((e = cudaMemsetAsync(base, 0, StaticLayout::header, st)) != cudaSuccess) return say(SOAP_ERR_CUDA, cudaGetErrorString(e));
    if ((e = cudaMemsetAsync(cell_count, 0, sizeof(int) * (kStaticMaxCells + 1), st)) != cudaSuccess) return say(SOAP_ERR_CUDA, cudaGetErrorString(e));
    bbox_only_kernel<<<blocks_for(N, 256, 256), 256, 0, st>>>(d_positions, N, g, bbox);
    grid_setup_kernel<<<1, 1, 0, st>>>(bbox, g, N, kStaticMaxCells, grid, nullptr);
    bin_count_kernel<<<blocks_for(N, 256), 256, 0, st>>>(d_positions, N, g, grid, atom_cell, atom_wrap, cell_count, counters);
    scan_kernel<int><<<1, 1024, 0, st>>>(cell_count, cell_start, kStaticMaxCells, nullptr, &grid->n_cells);
    bin_fill_kernel<<<blocks_for(N, 256), 256, 0, st>>>(d_positions, N, atom_cell, atom_wrap, cell_start, cell_count, s_pos, s_wrap);
    count_kernel<<<(unsigned)((N + 7) / 8), 256, 0, st>>>(d_positions, nullptr, N, g, grid, atom_cell, atom_wrap, cell_start, s_pos, s_wrap,
                                                         d_counts, counters);
    if ((e = cudaGetLastError()) != cudaSuccess) return say(SOAP_ERR_CUDA, cudaGetErrorString(e));
    return SOAP_OK;
}

int soap_profile(soap_t* h, int enable) {
    if (!h) return SOAP_ERR_INVALID_ARG;
    if (enable) {
        int rc = ensure_device(h);
        if (rc) return rc;
        for (cudaEvent_t& e : h->ev)
            if (!e) CU(cudaEventCreate(&e));
    }
    h->profiling = enable != 0;
    return SOAP_OK;
}

int soap_profile_read(soap_t* h, float* ms_neighbors, float* ms_center) {
    if (!h || !h->ev[2]) return SOAP_ERR_INVALID_ARG;
    CU(cudaEventSynchronize(h->ev[2]));
    float a = 0.f, b = 0.f;
    CU(cudaEventElapsedTime(&a, h->ev[0], h->ev[1]));
    CU(cudaEventElapsedTime(&b, h->ev[1], h->ev[2]));
    if (ms_neighbors) *ms_neighbors = a;
    if (ms_center) *ms_center = b;
    return SOAP_OK;
}

}  // extern "C"
