// Cell list and neighbour compaction (the search step under Eq. 1).
//
// Atoms are binned in fractional coordinates of the cell (of the identity when
// there is none); periodic axes are wrapped for binning only.  A centre visits
// the stencil of bins around its own, and every candidate (atom j, lattice
// translation n) passes the exact test
//     0 < |(r_j - r_i) + ((n_a a + n_b b) + n_c c)|^2 < r_cut^2
// in fp64 on the raw fp32 inputs, each operation rounded separately, so the set
// does not depend on the binning and can be compared bit for bit with a
// reference.  Pairs of a centre come out sorted by (atom, n_a, n_b, n_c).
#pragma once
#include "soap_device.cuh"

namespace soap {

// ---- order-preserving encoding of doubles for atomicMax ---------------------
__device__ inline unsigned long long enc_double(double x) {
    unsigned long long b = (unsigned long long)__double_as_longlong(x);
    return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}
__device__ inline double dec_double(unsigned long long e) {
    unsigned long long b = (e >> 63) ? (e & 0x7fffffffffffffffull) : ~e;
    return __longlong_as_double((long long)b);
}

__device__ inline void frac_coords(const Geometry& g, float x, float y, float z, double s[3]) {
    for (int a = 0; a < 3; ++a)
        s[a] = (double)x * g.inv[0 + a] + (double)y * g.inv[3 + a] + (double)z * g.inv[6 + a];
}

// species index per atom, and the bounding box of the fractional coordinates
// bbox[0..2] = enc(max s), bbox[3..5] = enc(max -s); zero-initialised by the host
__global__ void species_bbox_kernel(const float* __restrict__ pos, const int* __restrict__ numbers, long long N,
                                    Geometry geom, const int* __restrict__ z_lut, int* __restrict__ species_idx,
                                    unsigned long long* bbox, Counters* counters) {
    double hi[3] = {-1e300, -1e300, -1e300}, lo[3] = {-1e300, -1e300, -1e300};
    bool bad = false;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < N; i += (long long)gridDim.x * blockDim.x) {
        int z = numbers[i];
        int s = (z >= 0 && z < 128) ? z_lut[z] : -1;
        if (s < 0) { bad = true; s = 0; }
        species_idx[i] = s;
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
    if (bad) atomicOr(&counters->status, kStatusUnknownSpecies);
}

// One thread: choose the bin grid.  Bin width (measured perpendicular to the
// cell faces) is at least r_cut (1 + 1e-6) wherever more than one bin fits, so a
// stencil of +-1 bin covers the sphere; short periodic axes get one bin and a
// wider stencil of images.
__device__ inline GridParams choose_grid(const double hi_in[3], const double lo_in[3], const Geometry& geom, long long N, int cell_cap) {
    GridParams g;
    const double rc = geom.r_cut * (1.0 + 1e-6);
    double want[3];
    for (int a = 0; a < 3; ++a) {
        g.periodic[a] = geom.pbc[a];
        if (geom.pbc[a]) {
            g.smin[a] = 0.0;
            want[a] = floor(geom.height[a] / rc);
        } else {
            double hi = N > 0 ? hi_in[a] : 0.0, lo = N > 0 ? lo_in[a] : 0.0;
            g.smin[a] = lo;
            want[a] = floor((hi - lo) * geom.height[a] / rc);
        }
        if (!(want[a] >= 1.0)) want[a] = 1.0;
        if (want[a] > 1024.0) want[a] = 1024.0;
    }
    // respect the scratch capacity: shrink the grid uniformly
    for (int it = 0; it < 64 && want[0] * want[1] * want[2] > (double)cell_cap; ++it)
        for (int a = 0; a < 3; ++a) want[a] = fmax(1.0, floor(want[a] * 0.8));
    for (int a = 0; a < 3; ++a) {
        g.nb[a] = (int)want[a];
        if (geom.pbc[a]) {
            g.sscale[a] = (double)g.nb[a];
            double width = geom.height[a] / g.nb[a];
            g.R[a] = (int)ceil(rc / width);
        } else {
            double hi = N > 0 ? hi_in[a] : 0.0;
            double span = hi - g.smin[a];
            g.sscale[a] = span > 0 ? g.nb[a] / span : 0.0;
            g.R[a] = g.nb[a] > 1 ? 1 : 0;
        }
    }
    g.n_cells = g.nb[0] * g.nb[1] * g.nb[2];
    return g;
}

__global__ void grid_setup_kernel(const unsigned long long* bbox, Geometry geom, long long N, int cell_cap, GridParams* out,
                                  Counters* counters) {
    if (counters) { counters->n_pairs = 0; counters->n_rows = 0; }      // the pair cursor of this call
    double hi[3], lo[3];
    for (int a = 0; a < 3; ++a) { hi[a] = dec_double(bbox[a]); lo[a] = -dec_double(bbox[3 + a]); }
    *out = choose_grid(hi, lo, geom, N, cell_cap);
}

__device__ inline void bin_of(const Geometry& geom, const GridParams& g, float x, float y, float z, int b[3], int w[3]) {
    double s[3];
    frac_coords(geom, x, y, z, s);
    for (int a = 0; a < 3; ++a) {
        double t = s[a];
        w[a] = 0;
        if (g.periodic[a]) {
            double fl = floor(t);
            w[a] = (int)fl;
            t -= fl;
        }
        int bi = (int)floor((t - g.smin[a]) * g.sscale[a]);
        b[a] = min(max(bi, 0), g.nb[a] - 1);
    }
}

__device__ inline int pack3(const int v[3]) { return ((v[0] + 512) << 20) | ((v[1] + 512) << 10) | (v[2] + 512); }
__device__ inline void unpack3(int p, int v[3]) { v[0] = ((p >> 20) & 1023) - 512; v[1] = ((p >> 10) & 1023) - 512; v[2] = (p & 1023) - 512; }

__global__ void bin_count_kernel(const float* __restrict__ pos, long long N, Geometry geom, const GridParams* __restrict__ gp,
                                 int* __restrict__ atom_cell, int* __restrict__ atom_wrap, int* cell_count, Counters* counters) {
    const GridParams g = *gp;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < N; i += (long long)gridDim.x * blockDim.x) {
        int b[3], w[3];
        bin_of(geom, g, pos[3 * i], pos[3 * i + 1], pos[3 * i + 2], b, w);
        if (abs(w[0]) > 100 || abs(w[1]) > 100 || abs(w[2]) > 100) {      // positions absurdly far outside the cell
            atomicOr(&counters->status, kStatusShiftRange);
            w[0] = w[1] = w[2] = 0;
        }
        int cell = (b[2] * g.nb[1] + b[1]) * g.nb[0] + b[0];
        atom_cell[i] = cell;
        atom_wrap[i] = pack3(w);
        atomicAdd(&cell_count[cell], 1);
    }
}

// Exclusive scan by ONE block (n is at most a few million here); out[n] = total.
template <typename OutT>
__global__ void scan_kernel(const int* __restrict__ in, OutT* __restrict__ out, long long n, long long* total_out,
                            const int* n_dev = nullptr) {
    if (n_dev) n = min(n, (long long)*n_dev);          // only the bins the grid really uses
    __shared__ long long warp_sums[32];
    __shared__ long long carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    for (long long base = 0; base < n; base += blockDim.x) {
        long long i = base + threadIdx.x;
        long long v = i < n ? (long long)in[i] : 0, x = v;
        for (int o = 1; o < 32; o <<= 1) {
            long long y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if (lane == 31) warp_sums[wid] = x;
        __syncthreads();
        if (wid == 0) {
            long long s = lane < nw ? warp_sums[lane] : 0;
            for (int o = 1; o < 32; o <<= 1) {
                long long y = __shfl_up_sync(0xffffffffu, s, o);
                if (lane >= o) s += y;
            }
            warp_sums[lane] = s;
        }
        __syncthreads();
        long long carry = carry_s;
        long long excl = carry + (wid > 0 ? warp_sums[wid - 1] : 0) + x - v;
        if (i < n) out[i] = (OutT)excl;
        __syncthreads();
        if (threadIdx.x == blockDim.x - 1) carry_s = carry + warp_sums[nw - 1];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        out[n] = (OutT)carry_s;
        if (total_out) *total_out = carry_s;
    }
}

// Exclusive scan of long arrays in three launches: sums of tiles of kScanTile items, a one-block
// scan of those sums, then every tile scans itself on top of its offset.
constexpr int kScanTile = 4096;          // 1024 threads x 4 items
__global__ void __launch_bounds__(1024) tile_sum_kernel(const int* __restrict__ in, long long n, int* __restrict__ tile_sums) {
    __shared__ int ws[32];
    const long long base = (long long)blockIdx.x * kScanTile;
    int v = 0;
    for (int k = 0; k < 4; ++k) {
        const long long i = base + k * 1024 + threadIdx.x;
        if (i < n) v += in[i];
    }
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) ws[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x < 32) {
        int t = ws[threadIdx.x];
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (threadIdx.x == 0) tile_sums[blockIdx.x] = t;
    }
}
template <typename OutT>
__global__ void __launch_bounds__(1024) tile_scan_kernel(const int* __restrict__ in, OutT* __restrict__ out, long long n,
                                                         const long long* __restrict__ tile_offsets, long long n_tiles) {
    __shared__ long long ws[32];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const long long base = (long long)blockIdx.x * kScanTile + threadIdx.x * 4;      // 4 consecutive items per thread
    int v[4];
    long long mine = 0;
    for (int k = 0; k < 4; ++k) { v[k] = base + k < n ? in[base + k] : 0; mine += v[k]; }
    long long x = mine;
    for (int o = 1; o < 32; o <<= 1) {
        const long long y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += y;
    }
    if (lane == 31) ws[wid] = x;
    __syncthreads();
    if (wid == 0) {
        long long t = ws[lane];
        for (int o = 1; o < 32; o <<= 1) {
            const long long y = __shfl_up_sync(0xffffffffu, t, o);
            if (lane >= o) t += y;
        }
        ws[lane] = t;
    }
    __syncthreads();
    long long run = tile_offsets[blockIdx.x] + (wid > 0 ? ws[wid - 1] : 0) + x - mine;
    for (int k = 0; k < 4; ++k) {
        if (base + k < n) out[base + k] = (OutT)run;
        run += v[k];
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) out[n] = (OutT)tile_offsets[n_tiles];
}

__global__ void bin_fill_kernel(const float* __restrict__ pos, long long N, const int* __restrict__ atom_cell,
                                const int* __restrict__ atom_wrap, const int* __restrict__ cell_start, int* cell_count,
                                float4* __restrict__ s_pos, int* __restrict__ s_wrap) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < N; i += (long long)gridDim.x * blockDim.x) {
        int cell = atom_cell[i];
        int slot = cell_start[cell] + atomicSub(&cell_count[cell], 1) - 1;
        s_pos[slot] = make_float4(pos[3 * i], pos[3 * i + 1], pos[3 * i + 2], __int_as_float((int)i));
        s_wrap[slot] = atom_wrap[i];
    }
}

// Small structures: species lookup, bounding box, grid choice, binning, bin scan and the sort of
// the atoms by bin in ONE launch of a single CTA (five dependent launches otherwise; at a few
// thousand atoms the launches, not the work, set the time).
constexpr int kPrepThreads = 1024;
constexpr long long kSmallPrepAtoms = 16384;
constexpr int kPrepSmemCells = 4096;
__global__ void __launch_bounds__(kPrepThreads)
small_prep_kernel(const float* __restrict__ pos, const int* __restrict__ numbers, long long N, Geometry geom,
                  const int* __restrict__ z_lut, int* __restrict__ species_idx, int cell_cap, GridParams* grid_out,
                  int* __restrict__ atom_cell, int* __restrict__ atom_wrap, int* cell_count, int* cell_start,
                  float4* __restrict__ s_pos, int* __restrict__ s_wrap, Counters* counters) {
    __shared__ double red[6][32];
    __shared__ GridParams sg;
    __shared__ long long warp_sums[32];
    __shared__ long long carry_s;
    __shared__ int s_cnt[kPrepSmemCells + 1], s_start[kPrepSmemCells + 1];   // bin counters on chip when they fit
    grid_dependency_launch();                                                // the pair kernel may move in and wait
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    // ---- species and bounding box of the fractional coordinates ----
    double hi[3] = {-1e300, -1e300, -1e300}, lo[3] = {-1e300, -1e300, -1e300};
    bool bad = false;
    for (long long i = tid; i < N; i += kPrepThreads) {
        int z = numbers ? numbers[i] : 0;
        int s = numbers ? ((z >= 0 && z < 128) ? z_lut[z] : -1) : 0;
        if (s < 0) { bad = true; s = 0; }
        if (species_idx) species_idx[i] = s;
        double f[3];
        frac_coords(geom, pos[3 * i], pos[3 * i + 1], pos[3 * i + 2], f);
        for (int a = 0; a < 3; ++a) { hi[a] = fmax(hi[a], f[a]); lo[a] = fmax(lo[a], -f[a]); }
    }
    if (bad) atomicOr(&counters->status, kStatusUnknownSpecies);
    for (int a = 0; a < 3; ++a) {
        for (int o = 16; o > 0; o >>= 1) {
            hi[a] = fmax(hi[a], __shfl_xor_sync(0xffffffffu, hi[a], o));
            lo[a] = fmax(lo[a], __shfl_xor_sync(0xffffffffu, lo[a], o));
        }
        if (lane == 0) { red[a][wid] = hi[a]; red[3 + a][wid] = lo[a]; }
    }
    __syncthreads();
    if (wid == 0) {
        // the 32 warps' maxima, one per lane
        for (int a = 0; a < 6; ++a) {
            double v = red[a][lane];
            for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
            if (lane == 0) red[a][0] = v;
        }
    }
    __syncthreads();
    if (tid == 0) {
        double h3[3], l3[3];
        for (int a = 0; a < 3; ++a) { h3[a] = red[a][0]; l3[a] = -red[3 + a][0]; }
        sg = choose_grid(h3, l3, geom, N, cell_cap);
        *grid_out = sg;
        carry_s = 0;
        counters->n_pairs = 0;                                            // the pair cursor of this call
        counters->n_rows = 0;
    }
    __syncthreads();
    const GridParams g = sg;
    const bool on_chip = g.n_cells <= kPrepSmemCells;
    int* cnt = on_chip ? s_cnt : cell_count;
    // ---- bin counts ----
    for (int c = tid; c <= g.n_cells; c += kPrepThreads) cnt[c] = 0;
    __syncthreads();
    for (long long i = tid; i < N; i += kPrepThreads) {
        int b[3], w[3];
        bin_of(geom, g, pos[3 * i], pos[3 * i + 1], pos[3 * i + 2], b, w);
        if (abs(w[0]) > 100 || abs(w[1]) > 100 || abs(w[2]) > 100) {
            atomicOr(&counters->status, kStatusShiftRange);
            w[0] = w[1] = w[2] = 0;
        }
        const int cell = (b[2] * g.nb[1] + b[1]) * g.nb[0] + b[0];
        atom_cell[i] = cell;
        atom_wrap[i] = pack3(w);
        atomicAdd(&cnt[cell], 1);
    }
    __syncthreads();
    // ---- exclusive scan of the bin counts ----
    for (int base = 0; base < g.n_cells; base += kPrepThreads) {
        const int i = base + tid;
        const long long v = i < g.n_cells ? (long long)cnt[i] : 0;
        long long x = v;
        for (int o = 1; o < 32; o <<= 1) {
            const long long y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if (lane == 31) warp_sums[wid] = x;
        __syncthreads();
        if (wid == 0) {
            long long sacc = warp_sums[lane];
            for (int o = 1; o < 32; o <<= 1) {
                const long long y = __shfl_up_sync(0xffffffffu, sacc, o);
                if (lane >= o) sacc += y;
            }
            warp_sums[lane] = sacc;
        }
        __syncthreads();
        const long long carry = carry_s;
        if (i < g.n_cells) {
            const int st = (int)(carry + (wid > 0 ? warp_sums[wid - 1] : 0) + x - v);
            cell_start[i] = st;
            if (on_chip) s_start[i] = st;
        }
        __syncthreads();
        if (tid == kPrepThreads - 1) carry_s = carry + warp_sums[31];
        __syncthreads();
    }
    if (tid == 0) cell_start[g.n_cells] = (int)carry_s;
    __syncthreads();
    // ---- atoms sorted by bin ----
    const int* starts = on_chip ? s_start : cell_start;
    for (long long i = tid; i < N; i += kPrepThreads) {
        const int cell = atom_cell[i];
        const int slot = starts[cell] + atomicSub(&cnt[cell], 1) - 1;
        s_pos[slot] = make_float4(pos[3 * i], pos[3 * i + 1], pos[3 * i + 2], __int_as_float((int)i));
        s_wrap[slot] = atom_wrap[i];
    }
}

// floor division / modulo for the periodic wrap of a bin coordinate
__device__ inline void wrap_bin(int b, int nb, int& cell, int& image) {
    image = (b >= 0) ? b / nb : -((-b + nb - 1) / nb);
    cell = b - image * nb;
}

// Calls f(valid, key) for every lane in lock step, over all candidates of one centre.
// key encodes (atom, lattice translation on the raw inputs); valid says whether this
// lane holds a pair inside the cutoff.
// The stencil is walked 32 bins at a time: each lane fetches the atom range of one bin (a single
// memory round trip for all of them), a warp scan turns the counts into offsets, and the lanes
// then run over the concatenated candidates, so they stay busy whatever the bin occupancy.
template <class F>
__device__ inline void for_each_candidate(const Geometry& geom, const GridParams& g, const int* __restrict__ cell_start,
                                          const float4* __restrict__ s_pos, const int* __restrict__ s_wrap,
                                          float xi, float yi, float zi, const int bi[3], const int wi[3],
                                          int lane, Counters* counters, F f) {
    const int w0 = 2 * g.R[0] + 1, w1 = 2 * g.R[1] + 1, w2 = 2 * g.R[2] + 1;
    const int n_stencil = w0 * w1 * w2;
    const bool any_periodic = g.periodic[0] | g.periodic[1] | g.periodic[2];
    for (int q0 = 0; q0 < n_stencil; q0 += 32) {
        // ---- this lane's bin of the stencil ----
        const int q = q0 + lane;
        int start = 0, cnt = 0, img = 0;                  // img: packed image of the bin (periodic axes)
        if (q < n_stencil) {
            int o[3] = {q % w0 - g.R[0], (q / w0) % w1 - g.R[1], q / (w0 * w1) - g.R[2]};
            int c[3], im[3];
            bool inside = true;
            for (int a = 0; a < 3; ++a) {
                if (g.periodic[a]) wrap_bin(bi[a] + o[a], g.nb[a], c[a], im[a]);
                else { c[a] = bi[a] + o[a]; im[a] = 0; inside &= (c[a] >= 0 && c[a] < g.nb[a]); }
            }
            if (inside) {
                const int cell = (c[2] * g.nb[1] + c[1]) * g.nb[0] + c[0];
                start = cell_start[cell];
                cnt = cell_start[cell + 1] - start;
                img = pack3(im);
            }
        }
        // ---- offsets of the bins in the concatenated candidate list ----
        int incl = cnt;
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += y;
        }
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        for (int t0 = 0; t0 < total; t0 += 32) {
            const int t = t0 + lane;
            // bin of candidate t: the first lane whose inclusive offset exceeds t (binary search by shuffles)
            int lo = 0;
            for (int step = 16; step > 0; step >>= 1) {
                const int probe = __shfl_sync(0xffffffffu, incl, lo + step - 1);
                if (probe <= t) lo += step;
            }
            lo = min(lo, 31);
            const int b_incl = __shfl_sync(0xffffffffu, incl, lo), b_cnt = __shfl_sync(0xffffffffu, cnt, lo);
            const int b_start = __shfl_sync(0xffffffffu, start, lo), b_img = __shfl_sync(0xffffffffu, img, lo);
            bool valid = false;
            unsigned long long key = 0;
            if (t < total) {
                const int at = b_start + (t - (b_incl - b_cnt));
                const float4 pj = s_pos[at];
                int wj[3], im[3];
                unpack3(s_wrap[at], wj);
                unpack3(b_img, im);
                // translation on the raw (unwrapped) inputs
                const int na = im[0] - wj[0] + wi[0], nb = im[1] - wj[1] + wi[1], nc = im[2] - wj[2] + wi[2];
                double dx = __dsub_rn((double)pj.x, (double)xi);
                double dy = __dsub_rn((double)pj.y, (double)yi);
                double dz = __dsub_rn((double)pj.z, (double)zi);
                if (any_periodic) {
                    // T = (n_a a + n_b b) + n_c c, each product and sum rounded on its own
                    const double fa = (double)na, fb = (double)nb, fc = (double)nc;
                    double tx = __dadd_rn(__dadd_rn(__dmul_rn(fa, geom.cell[0]), __dmul_rn(fb, geom.cell[3])), __dmul_rn(fc, geom.cell[6]));
                    double ty = __dadd_rn(__dadd_rn(__dmul_rn(fa, geom.cell[1]), __dmul_rn(fb, geom.cell[4])), __dmul_rn(fc, geom.cell[7]));
                    double tz = __dadd_rn(__dadd_rn(__dmul_rn(fa, geom.cell[2]), __dmul_rn(fb, geom.cell[5])), __dmul_rn(fc, geom.cell[8]));
                    dx = __dadd_rn(dx, tx); dy = __dadd_rn(dy, ty); dz = __dadd_rn(dz, tz);
                }
                const double d2 = __dadd_rn(__dadd_rn(__dmul_rn(dx, dx), __dmul_rn(dy, dy)), __dmul_rn(dz, dz));
                valid = (d2 < geom.rc2) && (d2 > 0.0);
                if (valid && (abs(na) > 127 || abs(nb) > 127 || abs(nc) > 127)) {
                    atomicOr(&counters->status, kStatusShiftRange);
                    valid = false;
                }
                key = ((unsigned long long)(unsigned)__float_as_int(pj.w) << 24) |
                      ((unsigned long long)(na + 128) << 16) | ((unsigned long long)(nb + 128) << 8) |
                      (unsigned long long)(nc + 128);
            }
            f(valid, key);
        }
    }
}

// The same walk for the common case (no periodic axis, stencil of +-1 bin): the three bins of a stencil row along
// x are neighbours in the sorted atom array, so the 27 bins are 9 contiguous runs.  Every lane keeps the nine run
// boundaries in registers, and a candidate finds its run with compares instead of shuffles.
template <class F>
__device__ inline void for_each_candidate_runs(const Geometry& geom, const GridParams& g, const int* __restrict__ cell_start,
                                               const float4* __restrict__ s_pos, float xi, float yi, float zi,
                                               const int bi[3], int lane, F f) {
    // lane r < 9 fetches run r = (dy + 1) + 3 (dz + 1)
    int start = 0, cnt = 0;
    if (lane < 9) {
        const int cy = bi[1] + lane % 3 - g.R[1], cz = bi[2] + lane / 3 - g.R[2];
        const bool inside = cy >= 0 && cy < g.nb[1] && cz >= 0 && cz < g.nb[2] && (lane % 3 <= 2 * g.R[1]) && (lane / 3 <= 2 * g.R[2]);
        if (inside) {
            const int x0 = max(bi[0] - g.R[0], 0), x1 = min(bi[0] + g.R[0], g.nb[0] - 1);
            const int row = (cz * g.nb[1] + cy) * g.nb[0];
            start = cell_start[row + x0];
            cnt = cell_start[row + x1 + 1] - start;
        }
    }
    int r_start[9], r_end[9], total = 0;                 // run r covers candidates r_end[r] - count .. r_end[r] - 1
#pragma unroll
    for (int r = 0; r < 9; ++r) {
        const int c = __shfl_sync(0xffffffffu, cnt, r);
        r_start[r] = __shfl_sync(0xffffffffu, start, r) - total;      // atom index = r_start[r] + t for t inside run r
        total += c;
        r_end[r] = total;
    }
    for (int t0 = 0; t0 < total; t0 += 32) {
        const int t = t0 + lane;
        bool valid = false;
        unsigned long long key = 0;
        if (t < total) {
            int at = r_start[8];
#pragma unroll
            for (int r = 7; r >= 0; --r) at = t < r_end[r] ? r_start[r] : at;
            const float4 pj = s_pos[at + t];
            const double dx = __dsub_rn((double)pj.x, (double)xi);
            const double dy = __dsub_rn((double)pj.y, (double)yi);
            const double dz = __dsub_rn((double)pj.z, (double)zi);
            const double d2 = __dadd_rn(__dadd_rn(__dmul_rn(dx, dx), __dmul_rn(dy, dy)), __dmul_rn(dz, dz));
            valid = (d2 < geom.rc2) && (d2 > 0.0);
            key = ((unsigned long long)(unsigned)__float_as_int(pj.w) << 24) | 0x808080ull;
        }
        f(valid, key);
    }
}

// One warp per centre: number of pairs.
__global__ void count_kernel(const float* __restrict__ pos, const int* __restrict__ centers, long long C, Geometry geom,
                             const GridParams* __restrict__ gp, const int* __restrict__ atom_cell, const int* __restrict__ atom_wrap,
                             const int* __restrict__ cell_start, const float4* __restrict__ s_pos, const int* __restrict__ s_wrap,
                             int* __restrict__ pair_count, Counters* counters) {
    const GridParams g = *gp;
    const int lane = threadIdx.x & 31;
    const long long c = blockIdx.x * (long long)(blockDim.x >> 5) + (threadIdx.x >> 5);
    if (c >= C) return;
    const int i = centers ? centers[c] : (int)c;
    const float xi = pos[3 * (long long)i], yi = pos[3 * (long long)i + 1], zi = pos[3 * (long long)i + 2];
    int bi[3], wi[3];
    {
        int cell = atom_cell[i];
        bi[0] = cell % g.nb[0]; bi[1] = (cell / g.nb[0]) % g.nb[1]; bi[2] = cell / (g.nb[0] * g.nb[1]);
        unpack3(atom_wrap[i], wi);
    }
    int cnt = 0;
    for_each_candidate(geom, g, cell_start, s_pos, s_wrap, xi, yi, zi, bi, wi, lane, counters,
                       [&](bool valid, unsigned long long) { cnt += __popc(__ballot_sync(0xffffffffu, valid)); });
    if (lane == 0) pair_count[c] = cnt;
}

constexpr int kFillSmemKeys = 512;       // per warp; longer rows are sorted through global memory
constexpr int kFillSmemKeysSmall = 128;  // variant for structures with few pairs per centre: 4x less shared memory, more warps resident
constexpr int kFillWarps = 4;

// One warp per centre, one walk over the candidates: collect the pairs, reserve a segment of the
// pair arrays with one atomic add (segments follow the order in which warps arrive, so the pair
// arrays are addressed through pair_start / pair_count, not through a prefix sum), sort the keys,
// derive the Jacobian row bookkeeping (distinct atoms, the centre's own position among them).
// When the segment does not fit the planned capacity only the counts are produced and the status
// word says so; the caller plans again with the totals.
// ROWS = false (descriptor-only calls, which sum over the pairs in any order and have no Jacobian rows): the keys
// go out as they were found, unsorted, and the row bookkeeping is left out.
template <int KEYS, bool ROWS>
__global__ void __launch_bounds__(kFillWarps * 32)
pairs_kernel(const float* __restrict__ pos, const int* __restrict__ centers, const float* __restrict__ sites, long long C, Geometry geom,
             const GridParams* __restrict__ gp, const int* __restrict__ atom_cell, const int* __restrict__ atom_wrap,
             const int* __restrict__ cell_start, const float4* __restrict__ s_pos, const int* __restrict__ s_wrap,
             long long pair_capacity, unsigned long long* pair_tmp, unsigned long long* pair_key, int* __restrict__ pair_row,
             long long* __restrict__ pair_start, int* __restrict__ pair_count, int* __restrict__ row_count,
             int* __restrict__ self_row, Counters* counters) {
    __shared__ unsigned long long s_raw[kFillWarps][KEYS];
    __shared__ unsigned long long s_sorted[kFillWarps][KEYS];
    grid_dependency_launch();
    grid_dependency_wait();                                                  // the cell list of the kernel before
    const GridParams g = *gp;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const long long c = blockIdx.x * (long long)kFillWarps + wid;
    if (c >= C) return;
    // a centre is an atom, or (with `sites`) a point of its own: no atom index, no row of its own
    const bool site = sites != nullptr;
    const int i = site ? -1 : (centers ? centers[c] : (int)c);
    const float* pc = site ? sites + 3 * c : pos + 3 * (long long)i;
    const float xi = pc[0], yi = pc[1], zi = pc[2];
    int bi[3], wi[3];
    if (site) {
        bin_of(geom, g, xi, yi, zi, bi, wi);
        if (abs(wi[0]) > 100 || abs(wi[1]) > 100 || abs(wi[2]) > 100) {
            if (lane == 0) atomicOr(&counters->status, kStatusShiftRange);
            wi[0] = wi[1] = wi[2] = 0;
        }
    } else {
        int cell = atom_cell[i];
        bi[0] = cell % g.nb[0]; bi[1] = (cell / g.nb[0]) % g.nb[1]; bi[2] = cell / (g.nb[0] * g.nb[1]);
        unpack3(atom_wrap[i], wi);
    }
    // ---- walk the candidates; keep the keys on chip while they fit ----
    int k = 0;
    auto collect = [&](bool valid, unsigned long long key) {
        const unsigned m = __ballot_sync(0xffffffffu, valid);
        const int at = k + __popc(m & ((1u << lane) - 1));
        if (valid && at < KEYS) s_raw[wid][at] = key;
        k += __popc(m);
    };
    const bool runs = !(g.periodic[0] | g.periodic[1] | g.periodic[2]) && g.R[0] <= 1 && g.R[1] <= 1 && g.R[2] <= 1;
    if (runs) for_each_candidate_runs(geom, g, cell_start, s_pos, xi, yi, zi, bi, lane, collect);
    else for_each_candidate(geom, g, cell_start, s_pos, s_wrap, xi, yi, zi, bi, wi, lane, counters, collect);
    long long base = 0;
    if (lane == 0) base = (long long)atomicAdd(reinterpret_cast<unsigned long long*>(&counters->n_pairs), (unsigned long long)k);
    base = __shfl_sync(0xffffffffu, base, 0);
    const bool fits = base + k <= pair_capacity;
    const bool in_smem = k <= KEYS;
    if (lane == 0) { pair_start[c] = base; pair_count[c] = fits ? k : 0; }
    if (!fits) {
        if (lane == 0) {
            atomicOr(&counters->status, kStatusPairCapacity);
            row_count[c] = k + 1;                         // upper bound; exact once the plan fits
            self_row[c] = 0;
        }
        return;
    }
    if (!in_smem) {
        // rare: more pairs than the on-chip buffer holds; walk again, now with a place to put them
        int at0 = 0;
        for_each_candidate(geom, g, cell_start, s_pos, s_wrap, xi, yi, zi, bi, wi, lane, counters,
                           [&](bool valid, unsigned long long key) {
                               const unsigned m = __ballot_sync(0xffffffffu, valid);
                               const int at = at0 + __popc(m & ((1u << lane) - 1));
                               if (valid && at < k) pair_tmp[base + at] = key;
                               at0 += __popc(m);
                           });
    }
    volatile unsigned long long* raw = in_smem ? s_raw[wid] : pair_tmp + base;
    volatile unsigned long long* sorted = in_smem ? s_sorted[wid] : pair_key + base;
    __syncwarp();
    if (!ROWS) {
        for (int q = lane; q < k; q += 32) pair_key[base + q] = raw[q];
        return;
    }
    // rank sort (keys are distinct), two keys per lane and trip so that every key read serves two comparisons;
    // without a periodic axis all keys carry the same lattice translation and the atom fields alone decide
    bool self_in = false;
    const bool atoms_only = !(geom.pbc[0] | geom.pbc[1] | geom.pbc[2]);
    for (int q = lane; q < k; q += 64) {
        const bool two = q + 32 < k;
        const unsigned long long key0 = raw[q], key1 = two ? raw[q + 32] : ~0ull;
        int rank0 = 0, rank1 = 0;
        if (atoms_only) {
            const unsigned a0 = (unsigned)(key0 >> 24), a1 = (unsigned)(key1 >> 24);
            for (int r = 0; r < k; ++r) {
                const unsigned a = (unsigned)(raw[r] >> 24);
                rank0 += a < a0; rank1 += a < a1;
            }
        } else {
            for (int r = 0; r < k; ++r) {
                const unsigned long long v = raw[r];
                rank0 += v < key0; rank1 += v < key1;
            }
        }
        sorted[rank0] = key0;
        if (in_smem) pair_key[base + rank0] = key0;
        self_in |= key_atom(key0) == i;
        if (two) {
            sorted[rank1] = key1;
            if (in_smem) pair_key[base + rank1] = key1;
            self_in |= key_atom(key1) == i;
        }
    }
    self_in = __any_sync(0xffffffffu, self_in);
    __syncwarp();
    // distinct atoms -> local Jacobian rows; the centre's own row sits in atom order
    int uniq = 0, below = 0;
    for (int q0 = 0; q0 < k; q0 += 32) {
        const int q = q0 + lane;
        int atom = -1, prev = -2;
        if (q < k) {
            atom = key_atom(sorted[q]);
            prev = q > 0 ? key_atom(sorted[q - 1]) : -1;
        }
        const bool isnew = q < k && atom != prev;
        const unsigned m = __ballot_sync(0xffffffffu, isnew);
        const int u = uniq + __popc(m & ((1u << lane) - 1)) + (isnew ? 1 : 0) - 1;   // index among distinct atoms
        if (q < k) {
            int row = u + ((!site && !self_in && atom > i) ? 1 : 0);
            if (!isnew) row |= kRowContinuation;
            if (atom == i) row |= kRowSelfImage;
            pair_row[base + q] = row;
        }
        below += __popc(__ballot_sync(0xffffffffu, isnew && atom < i));
        uniq += __popc(m);
    }
    if (lane == 0) {
        row_count[c] = uniq + ((site || self_in) ? 0 : 1);
        self_row[c] = site ? -1 : below;
    }
}

// Many independent non-periodic structures in one launch: atoms of all structures in one list,
// struct_ptr[b] .. struct_ptr[b+1]-1 the atoms of structure b, every atom a centre that sees only its own
// structure.  One warp per centre runs over the atoms of its structure (brute force: the structures
// this is for are small molecules, where the cutoff sphere holds most of the structure anyway), with the same
// exact fp64 test as the cell-list path; neighbours come out in ascending atom order, so nothing is sorted.
// Writes what pairs_kernel writes (keys with zero lattice translation) plus the species index of the centre.
__global__ void __launch_bounds__(kFillWarps * 32)
batch_pairs_kernel(const float* __restrict__ pos, const int* __restrict__ numbers, const int* __restrict__ z_lut,
                   int* __restrict__ species_idx, const long long* __restrict__ struct_ptr, long long n_structs,
                   long long N, double rc2, long long pair_capacity, unsigned long long* pair_key,
                   int* __restrict__ pair_row, long long* __restrict__ pair_start, int* __restrict__ pair_count,
                   int* __restrict__ row_count, int* __restrict__ self_row, Counters* counters) {
    grid_dependency_launch();
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const long long i = blockIdx.x * (long long)kFillWarps + wid;
    if (i >= N) return;
    if (lane == 0) {
        const int z = numbers[i];
        int s = (z >= 0 && z < 128) ? z_lut[z] : -1;
        if (s < 0) { atomicOr(&counters->status, kStatusUnknownSpecies); s = 0; }
        species_idx[i] = s;
    }
    // the structure that holds atom i: last b with struct_ptr[b] <= i (no offsets: one structure, all atoms)
    long long a = 0, b = N;
    if (struct_ptr) {
        long long lo = 0, hi = n_structs;
        while (hi - lo > 1) {
            const long long mid = (lo + hi) >> 1;
            if (struct_ptr[mid] <= i) lo = mid; else hi = mid;
        }
        a = struct_ptr[lo];
        b = min(struct_ptr[lo + 1], N);
    }
    const double xi = pos[3 * i], yi = pos[3 * i + 1], zi = pos[3 * i + 2];
    auto inside = [&](long long j) {
        if (j >= b) return false;
        const double dx = __dsub_rn((double)pos[3 * j], xi), dy = __dsub_rn((double)pos[3 * j + 1], yi),
                     dz = __dsub_rn((double)pos[3 * j + 2], zi);
        const double d2 = __dadd_rn(__dadd_rn(__dmul_rn(dx, dx), __dmul_rn(dy, dy)), __dmul_rn(dz, dz));
        return d2 < rc2 && d2 > 0.0;
    };
    int k = 0, below = 0;
    for (long long j0 = a; j0 < b; j0 += 32) {
        const bool v = inside(j0 + lane);
        k += __popc(__ballot_sync(0xffffffffu, v));
        below += __popc(__ballot_sync(0xffffffffu, v && j0 + lane < i));
    }
    long long base = 0;
    if (lane == 0) base = (long long)atomicAdd(reinterpret_cast<unsigned long long*>(&counters->n_pairs), (unsigned long long)k);
    base = __shfl_sync(0xffffffffu, base, 0);
    const bool fits = base + k <= pair_capacity;
    if (lane == 0) {
        pair_start[i] = base;
        pair_count[i] = fits ? k : 0;
        row_count[i] = k + 1;                     // the neighbours and the centre itself
        self_row[i] = below;
        if (!fits) atomicOr(&counters->status, kStatusPairCapacity);
    }
    if (!fits) return;
    int at = 0;
    for (long long j0 = a; j0 < b; j0 += 32) {
        const long long j = j0 + lane;
        const bool v = inside(j);
        const unsigned m = __ballot_sync(0xffffffffu, v);
        if (v) {
            const int q = at + __popc(m & ((1u << lane) - 1));
            pair_key[base + q] = ((unsigned long long)j << 24) | (128ull << 16) | (128ull << 8) | 128ull;
            pair_row[base + q] = q + (j > i ? 1 : 0);        // rows in atom order, the centre's own among them
        }
        at += __popc(m);
    }
}

// One block: exclusive scan of the row counts (rows of centre c start at row_ptr[c]) and the launch
// order of the per-centre kernel, largest pair count first (bins of 4 pairs, counting sort), so that
// the long CTAs do not end up alone at the tail of the launch.
constexpr int kSizeBins = 256, kSizeBinShift = 2;
__global__ void __launch_bounds__(1024)
rows_order_kernel(const int* __restrict__ row_count, const int* __restrict__ pair_count, long long C,
                  long long* __restrict__ row_ptr, int* __restrict__ order, Counters* counters) {
    __shared__ long long warp_sums[32];
    __shared__ long long carry_s;
    __shared__ int hist[kSizeBins], first_slot[kSizeBins];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    grid_dependency_launch();
    if (tid == 0) carry_s = 0;
    if (tid < kSizeBins) hist[tid] = 0;
    grid_dependency_wait();                                                  // the counts of the pair kernel
    __syncthreads();
    // four consecutive centres per thread and trip: a few thousand centres are one trip, four barriers
    constexpr int kPerThread = 4;
    for (long long base = 0; base < C; base += 1024 * kPerThread) {
        const long long i0 = base + (long long)tid * kPerThread;
        long long v[kPerThread], x = 0;
#pragma unroll
        for (int k = 0; k < kPerThread; ++k) {
            const long long i = i0 + k;
            v[k] = i < C ? (long long)row_count[i] : 0;
            if (i < C) atomicAdd(&hist[min(pair_count[i] >> kSizeBinShift, kSizeBins - 1)], 1);
            x += v[k];
        }
        const long long mine = x;
        for (int o = 1; o < 32; o <<= 1) {
            const long long y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if (lane == 31) warp_sums[wid] = x;
        __syncthreads();
        if (wid == 0) {
            long long sacc = warp_sums[lane];
            for (int o = 1; o < 32; o <<= 1) {
                const long long y = __shfl_up_sync(0xffffffffu, sacc, o);
                if (lane >= o) sacc += y;
            }
            warp_sums[lane] = sacc;
        }
        __syncthreads();
        const long long carry = carry_s;
        long long at = carry + (wid > 0 ? warp_sums[wid - 1] : 0) + x - mine;
#pragma unroll
        for (int k = 0; k < kPerThread; ++k) {
            if (i0 + k < C) row_ptr[i0 + k] = at;
            at += v[k];
        }
        __syncthreads();
        if (tid == 1023) carry_s = carry + warp_sums[31];
        __syncthreads();
    }
    if (tid == 0) {
        row_ptr[C] = carry_s;
        counters->n_rows = carry_s;
    }
    if (wid == 0) {
        // first slot of every size bin, largest bin first: lane k scans the bins 255 - 8k down to 248 - 8k, a warp
        // scan adds what the lanes before it hold
        constexpr int per_lane = kSizeBins / 32;
        const int top = kSizeBins - 1 - lane * per_lane;
        int mine = 0;
        for (int k = 0; k < per_lane; ++k) mine += hist[top - k];
        int incl = mine;
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += y;
        }
        int run = incl - mine;
        for (int k = 0; k < per_lane; ++k) { first_slot[top - k] = run; run += hist[top - k]; }
    }
    __syncthreads();
    if (order)
        for (long long i = tid; i < C; i += 1024) {
            const int b = min(pair_count[i] >> kSizeBinShift, kSizeBins - 1);
            order[atomicAdd(&first_slot[b], 1)] = (int)i;
        }
}

// Compact copy of the pair list (the pair arrays are addressed by segment): one warp per centre.
__global__ void export_pairs_kernel(const long long* __restrict__ pair_start, const long long* __restrict__ out_ptr,
                                    const unsigned long long* __restrict__ pair_key, long long C, long long capacity,
                                    int* out_atom, int* out_shift, Counters* counters) {
    if (out_ptr[C] > capacity) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(&counters->status, kStatusPairCapacity);
        return;
    }
    const int lane = threadIdx.x & 31;
    for (long long c = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5; c < C; c += ((long long)gridDim.x * blockDim.x) >> 5) {
        const long long src = pair_start[c], dst = out_ptr[c];
        const int k = (int)(out_ptr[c + 1] - dst);
        for (int q = lane; q < k; q += 32) {
            const unsigned long long key = pair_key[src + q];
            out_atom[dst + q] = key_atom(key);
            if (out_shift) {
                int sft[3];
                key_shift(key, sft);
                out_shift[3 * (dst + q)] = sft[0]; out_shift[3 * (dst + q) + 1] = sft[1]; out_shift[3 * (dst + q) + 2] = sft[2];
            }
        }
    }
}

}  // namespace soap
