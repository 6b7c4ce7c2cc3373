// Device-side data structures shared by the neighbour kernels and the fused
// per-centre kernel.  sm_100a only.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace soap {

constexpr int kMaxSpecies = 8;
constexpr int kThreads = 256;            // CTA size of the per-centre kernels
constexpr int kWarps = kThreads / 32;
constexpr int kMaxElemPerThread = 8;     // n_max (l_max+1)^2 / kThreads rounded up: 16*169/256 -> 11 is refused at create
constexpr int kMaxChanRounds = 7;        // n_max (l_max+1) / 32 rounded up: 16*13/32

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
    const int* species_idx;       // [N]
    long long n_centers;
    Geometry geom;
    // neighbour data
    const long long* pair_ptr;    // [C+1]
    const unsigned long long* pair_key;
    const int* pair_row;
    const long long* row_ptr;     // [C+1]
    const int* self_row;          // [C]
    long long pair_capacity, row_capacity;
    Counters* counters;
    // basis
    const float* table;           // [nint][n_ch][6]
    const float* self_term;       // [n_max]
    const float* anorm;
    const float* dfact;
    const float* kl;
    const int* feat_pack;         // [F] n | n'<<5 | mu<<10 | nu<<14 | l<<18
    float inv_h;
    int n_intervals;
    int S, n_max, l_max, F;
    int P;                        // pairs per chunk (multiple of 4, <= 32)
    // outputs
    float* out_desc;              // [C,F]
    float* out_jac;               // [rows,3,F]
    int* row_atom;                // [rows]
};

__host__ __device__ inline int key_atom(unsigned long long k) { return (int)(k >> 24); }
__host__ __device__ inline void key_shift(unsigned long long k, int s[3]) {
    s[0] = (int)((k >> 16) & 255) - 128;
    s[1] = (int)((k >> 8) & 255) - 128;
    s[2] = (int)(k & 255) - 128;
}

// Shared-memory carve-up of the per-centre kernel, in 4-byte words.
struct SmemLayout {
    int c, D, sd, sinfo, sSD, sG, sQ, sCS, sUV, total;
};
__host__ __device__ inline SmemLayout make_layout(int S, int n_max, int l_max, int P, bool deriv) {
    const int L1 = l_max + 1, LM = L1 * L1, NCH = n_max * L1, CT = S * n_max * LM;
    SmemLayout o;
    int off = 0;                                   // every region starts on a 16-byte boundary
    o.c = off; off = (off + CT + 3) & ~3;
    o.sd = off; off += P * 4;
    o.sinfo = off; off = (off + P * 2 + 3) & ~3;
    o.sSD = off; off = (off + (deriv ? P * LM * 4 : P * LM) + 3) & ~3;
    o.sG = off; off = (off + (deriv ? P * NCH * 2 : P * NCH) + 3) & ~3;
    o.sQ = off; off = (off + P * (L1 * (L1 + 1) / 2) + 3) & ~3;
    o.sCS = off; off = (off + P * L1 * 2 + 3) & ~3;
    // the D tiles (pass 1) and the U/V staging (pass 2) never live at the same time
    o.D = off; o.sUV = off;
    if (deriv) {
        int a = 3 * CT, b = P * S * NCH * 4;
        off += a > b ? a : b;
    }
    o.total = off;
    return o;
}

}  // namespace soap
