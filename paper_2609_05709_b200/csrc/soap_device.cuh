// Device-side data structures shared by the neighbour kernels and the fused
// per-centre kernel.  sm_100a only.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace soap {

constexpr int kMaxSpecies = 8;
constexpr int kThreads = 256;            // CTA size of the per-centre kernels
constexpr int kWarps = kThreads / 32;
constexpr int kMaxElemPerThread = 8;     // soap_create refuses n_max (l_max+1)^2 > 8 * kThreads (shared-memory budget of the tiles)

// status bits (device, sticky until soap_status)
constexpr int kStatusUnknownSpecies = 1;
constexpr int kStatusPairCapacity = 2;
constexpr int kStatusRowCapacity = 4;
constexpr int kStatusShiftRange = 8;

// pair_row flags
constexpr int kRowContinuation = 1 << 30;   // same atom (another image) as the previous pair
constexpr int kRowSelfImage = 1 << 29;      // a periodic image of the centre itself
constexpr int kRowMask = (1 << 29) - 1;

struct Geometry {                 // host-known, passed by value
    double cell[9];               // rows a, b, c (identity when no cell)
    double inv[9];                // inverse: frac = pos * inv
    double height[3];             // distance between opposite cell faces
    double r_cut, rc2;
    int pbc[3];
};

struct GridParams {               // device-resident, written by grid_setup_kernel
    int nb[3];                    // bins per axis
    int R[3];                     // stencil half-width in bins
    int periodic[3];
    double smin[3];               // bin = (s - smin) * sscale
    double sscale[3];
    int n_cells;
};

struct Counters {                 // device-resident
    int status;
    int pad;
    long long n_pairs;
    long long n_rows;
};

struct CenterParams {
    // structure
    const float* pos;             // [N,3]
    const int* centers;           // [C] or null
    const float* sites;           // [C,3] or null: centres at these points instead of at atoms (no on-site term, no own row)
    const int* order;             // [C] CTA -> centre slot (largest first) or null
    const int* species_idx;       // [N]
    long long n_centers;
    Geometry geom;
    // neighbour data
    const long long* pair_start;  // [C] first pair of the centre's segment
    const int* pair_count;        // [C]
    const unsigned long long* pair_key;
    const int* pair_row;
    const long long* row_ptr;     // [C+1]
    const int* self_row;          // [C]
    long long pair_capacity, row_capacity;
    Counters* counters;
    // basis
    const float* table;           // [nint][n_ch][6]
    const float* table_ln;        // the same polynomials as [nint][l][n / 2][6][2], n padded to a multiple of 4 (descriptor-only kernel)
    const float* self_term;       // [n_max]
    const int* l_of_lm;           // [lm] -> l
    const float* kl;
    const int* feat_pack;         // [F] n | n'<<5 | mu<<10 | nu<<14 | l<<18
    double inv_h;                 // intervals per Angstrom of the radial table in use
    int n_intervals;
    int S, n_max, l_max, F;
    int P;                        // pairs per staged chunk (<= 32)
    unsigned nch_magic;           // floor(2^32 / (n_max (l_max+1))) + 1: x / n_ch == umulhi(x, magic) for x < 65536
    // output mode
    int crossover;                // 0: only the species pairs mu == nu are features
    int emit_coeff;               // descriptor build: write the coefficients c^mu_nlm instead of the power spectrum
    const float* c_bar;           // [S n_max (l_max+1)^2] or null: coefficients that replace the centre's own after pass 1
    // inner average over ALL atoms as centres: the kernel writes, for its atom a, d pbar / d r_a = own_scale times the
    // contraction of cbar with sum_i grad_a c(i) (pass 1 collects that sum) to out_jac[a], and no per-pair rows
    int inner_rows;
    float own_scale;
    // outer average over ALL atoms as centres: coefficients of every centre, [C][S n_max (l_max+1)^2] (index
    // (mu n_max + n) (l_max+1)^2 + l^2 + l + m, on-site terms included); the kernel of atom a adds to its own row
    // the rows that the centres it sees hold for it, all times own_scale, in out_jac[a]
    const float* c_all;
    // species-compact Jacobian rows: a neighbour's row holds only the blocks that involve its species (pitch Fc, a
    // multiple of 8 floats); the centre's own full row goes to out_center [C,3,F]
    int compact, Fc;
    float* out_center;
    // radial weighting of the neighbour density: per pair (w(d), w'(d)/d), null when off; w0 scales the on-site term
    const float2* pair_w;
    float w0;
    // outputs
    float* out_desc;              // [C,F]  (coefficient mode: [C, S n_max (l_max+1)^2]; with c_bar: [F])
    float* out_jac;               // [rows,3,F]  (coefficient mode: [rows, 3, S n_max (l_max+1)^2])
    int* row_atom;                // [rows]
};

// Programmatic dependent launch: a kernel launched with the attribute cudaLaunchAttributeProgrammaticStreamSerialization
// may start while the kernel before it in the stream still runs; it must call grid_dependency_wait() before it
// touches anything that kernel (or one before it) wrote - the wait returns once that kernel has finished and its
// writes are visible (at once when the launch carried no attribute).  grid_dependency_launch() lets the NEXT kernel
// of the stream start; without it that happens when this kernel's blocks exit.
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// launch of a kernel that begins with grid_dependency_wait(), allowed to overlap the tail of its predecessor
template <class... KArgs, class... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

__host__ __device__ inline int key_atom(unsigned long long k) { return (int)(k >> 24); }
__host__ __device__ inline void key_shift(unsigned long long k, int s[3]) {
    s[0] = (int)((k >> 16) & 255) - 128;
    s[1] = (int)((k >> 8) & 255) - 128;
    s[2] = (int)(k & 255) - 128;
}

// Shared-memory carve-up of the per-centre kernel, in 4-byte words.  Every region
// starts on a 16-byte boundary.  Rows of the coefficient tiles and of the harmonics
// staging have the odd stride (l_max+1)^2 | 1, which keeps strided accesses off a
// single bank.
constexpr int kGeoPairs = 128;           // pairs whose geometry is staged at once

constexpr int kZeroWords = 1024;         // a block of zeros that bulk copies write into the structural-zero blocks of the rows

struct SmemLayout {
    int c, geo, tri, xdec, zero, D, wUV, sSD, sG, total;
};
// whether the cross-species blocks of the rows are written in table-driven sweeps (a decode table in shared
// memory): several species, n_max from 9 to 12 and n_max (l_max+1) not a multiple of four (the other cases have
// faster paths with an operand in registers)
__host__ __device__ inline bool cross_table_wanted(int S, int n_max, int l_max) {
    return S > 1 && n_max > 8 && n_max <= 12 && ((n_max * (l_max + 1)) & 3) != 0;
}
__host__ __device__ inline int align4(int x) { return (x + 3) & ~3; }
constexpr int kGeoWords = kGeoPairs * 9 + 44;   // geometry (9 words per pair), species segments (9 + 32 words, padded)
__host__ __device__ inline SmemLayout make_layout(int S, int n_max, int l_max, int P, bool deriv, bool weighted = false) {
    const int L1 = l_max + 1, LMP = (L1 * L1) | 1, NCH = n_max * L1, CT = S * n_max * LMP;
    SmemLayout o;
    int off = 0;
    o.c = off; off = align4(off + CT);
    o.geo = off; off = align4(off + kGeoWords + (weighted ? 2 * kGeoPairs : 0));   // + per-pair weights
    o.tri = off; if (deriv) off = align4(off + ((n_max * (n_max + 1) / 2) * L1 + 1) / 2);   // 16-bit entries
    o.xdec = off; if (deriv && cross_table_wanted(S, n_max, l_max)) off = align4(off + (n_max * NCH + 1) / 2);   // 16-bit entries
    o.zero = off; if (deriv) off += kZeroWords;
    // the D tiles (pass 1, centre's row) and the per-warp U/V staging (pass 2) never live
    // at the same time and share space
    o.D = off; o.wUV = off;
    if (deriv) {
        const int a = 3 * CT, b = kWarps * S * NCH * 4;
        off = align4(off + (a > b ? a : b));
    }
    o.sSD = off; off = align4(off + (deriv ? P * LMP * 4 : P * LMP));
    o.sG = off; off = align4(off + (deriv ? P * NCH * 2 : P * NCH));
    o.total = off;
    return o;
}

}  // namespace soap
