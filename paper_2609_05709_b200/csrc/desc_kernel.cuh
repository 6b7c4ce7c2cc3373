// The descriptor-only kernel: expansion coefficients (Eq. 13 / Eqs. 18-19) and the power spectrum
// (Eq. 4) of every centre, one WARP per centre, persistent CTAs whose warps take the centres in turn.
//
// This build is bound by FP32 issue slots and by shared-memory bandwidth, not by HBM, so the layout is
// chosen for few instructions and few shared-memory wavefronts per pair:
//   * the radial table (value polynomials, re-laid as [interval][l][n / 2][6][2]) sits in shared memory
//     once per CTA when it fits; a lane evaluates two adjacent n at once from three conflict-free 16-byte
//     loads and five packed multiply-adds (fma.rn.f32x2: one issue slot for two multiply-adds);
//   * the pairs of a centre (up to 64 at a time) have their geometry formed in registers, are ranked by species with ballots, and staged 16 at a time in
//     species order: solid
//     harmonics with a lane per pair from the fully unrolled Q_l^m recursion, radial factors with
//     lanes on the channels (l, n);
//   * accumulation c[l,m][n] += S_lm G_nl is register-tiled: a lane owns four consecutive m of one l
//     times all n (an outer product of 4 x n_max per pair from one 16-byte load of S and n_max/4 of
//     G); with at most 16 such tiles the two half-warps work on two pairs at once.  Sums stay in
//     registers over all pairs of a species and are added to the centre's tile c[lm][species, n]
//     once per species; the staging rows are laid out so that all these loads are conflict-free;
//   * Eq. 4 is the Gram matrix of that tile per l: lanes take 4 x 4 blocks of (species, n) pairs,
//     two 16-byte loads per 16 multiply-adds, and the feature row is put together in shared memory
//     and written out in order.
// Nothing but the pair list is read from HBM and nothing but the descriptor row is written.
#pragma once
#include "soap_device.cuh"

namespace soap {

constexpr int kDescChunk = 16;                    // pairs staged at once by a warp
constexpr int kDescGroup = 64;                    // pairs whose geometry a warp holds in registers (two per lane)
constexpr int kDescMaxWarps = 16;                 // warps per CTA (one CTA per SM)

// harmonic normalisation up to l = 12, filled by desc_constants(): a_lm (sqrt2 folded in for m > 0), index l(l+1)/2 + m
__device__ __constant__ float kd_norm[91] = {0};

// tiles of four consecutive m of one l: tile index of the first tile of row l, and their number up to l_max
__host__ __device__ constexpr int desc_tile_base(int l) {
    int t = 0;
    for (int k = 0; k < l; ++k) t += (2 * k + 1 + 3) / 4;
    return t;
}
__host__ __device__ constexpr int desc_tiles(int l_max) { return desc_tile_base(l_max + 1); }
// n_max is padded to a multiple of four (NP = 4, 8, 12 or 16 is the template parameter; the padding channels have
// all-zero table rows, so they cost arithmetic but need no special cases)
__host__ __device__ constexpr int desc_np(int n_max) { return (n_max + 3) & ~3; }
// words per pair of the harmonics staging: the tiles, four words each, padded to an odd number of 16-byte chunks so
// that the 16-byte stores of eight lanes (eight pairs) fall into eight different bank groups
__host__ __device__ constexpr int desc_s_row(int l_max) { return 4 * (desc_tiles(l_max) | 1); }
// words per l of the radial staging.  Lanes that own tiles of different l read 16-byte chunks of different rows at
// once, and these must fall into different bank groups: with an odd number of chunks per l they do; with two
// (n_max up to 8) the two chunks of rows l >= 4 are swapped instead; with four the row is padded by one chunk.
__host__ __device__ constexpr int desc_g_l(int np) { return np == 16 ? 20 : np; }
__host__ __device__ constexpr int desc_g_swap(int np, int l) { return np == 8 ? (l >> 2) & 1 : 0; }

// 16-byte chunks per row of the centre's coefficient tile c[lm][species, n]: S NP / 4 rounded up to a power of two.
// Chunk k of row r sits at position (k + r / 4) mod that number, so that the lanes of a warp, which own rows four
// apart, do not all hit one group of banks when they store their sums.
__host__ __device__ constexpr int desc_c_chunks(int S, int np) {
    int rc = 1;
    while (rc < S * np / 4) rc <<= 1;
    return rc;
}

// Shared memory in 4-byte words: [table (optional)] then one region per warp:
//   c [LM][4 desc_c_chunks] | S staging [chunk][s_row] | G staging [chunk][L1 g_l] | pair staging [chunk][8 or 5]
// The feature row is assembled on top of the staging area when it fits there.  With the table in shared memory (the
// plain build on many centres) a staged pair is five words (dx, dy, dz, t; interval | species << 16) instead of
// eight (dx, dy, dz, r; interval, t, species, weight): at the benchmark's basis that is what lets a 16th warp fit.
struct DescLayout {
    int table, warp0, per_warp, c, sS, sG, ring, slab_words, total;
};
__host__ __device__ inline DescLayout make_desc_layout(int S, int np, int l_max, int warps, int table_words) {
    const int L1 = l_max + 1, LM = L1 * L1;
    DescLayout o;
    o.table = 0;
    o.warp0 = (table_words + 3) & ~3;
    int off = 0;
    o.c = off; off += LM * 4 * desc_c_chunks(S, np);
    o.sS = off; off += kDescChunk * desc_s_row(l_max);
    o.sG = off; off += kDescChunk * L1 * desc_g_l(np);
    o.ring = off; off += kDescChunk * (table_words ? 5 : 8);
    off = (off + 3) & ~3;
    o.slab_words = off - o.sS;
    o.per_warp = off;
    o.total = o.warp0 + warps * off;
    return o;
}

// Real solid harmonics S_lm(d) = r^l Y_lm of one displacement, every (l, m), written as 16-byte tiles: tile
// desc_tile_base(l) + j holds m = 4j - l .. 4j + 3 - l of row l (zeros beyond m = l):
//   S_{l,+m} = a_lm Q_l^m Re (x+iy)^m,  S_{l,-m} = a_lm Q_l^m Im (x+iy)^m,
//   Q_m^m = (2m-1)!!,  (l+1-m) Q_{l+1}^m = (2l+1) z Q_l^m - (l+m) r^2 Q_{l-1}^m.
// Fully unrolled: every index is an immediate and the Q's live in registers.
template <int L>
__device__ __forceinline__ void harmonics_tiles(float x, float y, float z, float r2, float4* __restrict__ out) {
    float cm[L + 1], sm[L + 1];                   // (x+iy)^m
    cm[0] = 1.f; sm[0] = 0.f;
#pragma unroll
    for (int m = 1; m <= L; ++m) {
        cm[m] = x * cm[m - 1] - y * sm[m - 1];
        sm[m] = x * sm[m - 1] + y * cm[m - 1];
    }
    float q1[L + 1], q2[L + 1];                   // Q_l^m and Q_{l-1}^m while the loop is at l
#pragma unroll
    for (int m = 0; m <= L; ++m) { q1[m] = 0.f; q2[m] = 0.f; }
    float dfact = 1.f;                            // (2l-1)!!
#pragma unroll
    for (int l = 0; l <= L; ++l) {
        if (l > 0) dfact *= (float)(2 * l - 1);
        const float zl = (float)(2 * l - 1) * z;
        float row[2 * L + 4];                     // S_{l,m} at index m + l
#pragma unroll
        for (int i = 0; i < 2 * L + 4; ++i) row[i] = 0.f;
#pragma unroll
        for (int m = 0; m <= l; ++m) {
            float q;
            if (m == l) q = dfact;
            else q = (zl * q1[m] - (float)(l - 1 + m) * r2 * q2[m]) * (1.f / (float)(l - m));
            q2[m] = q1[m];
            q1[m] = q;
            const float aq = kd_norm[l * (l + 1) / 2 + m] * q;
            row[l + m] = aq * cm[m];
            if (m) row[l - m] = aq * sm[m];
        }
#pragma unroll
        for (int j = 0; j < (2 * l + 4) / 4; ++j)
            out[desc_tile_base(l) + j] = make_float4(row[4 * j], row[4 * j + 1], row[4 * j + 2], row[4 * j + 3]);
    }
}

// NP: n_max rounded up to a multiple of four.  PLAIN: the default configuration (atom centres, no weighting, every
// species pair, power spectrum out).  TS: the radial table is in shared memory.
template <int L, int NP, bool PLAIN, bool TS>
__global__ void __launch_bounds__(kDescMaxWarps * 32, 1) desc_kernel(const CenterParams p) {
    constexpr int L1 = L + 1, LM = L1 * L1;
    constexpr int NCHP = L1 * NP;                                        // channels (l, n), n padded
    constexpr int SROW = desc_s_row(L), GL = desc_g_l(NP), GROW = L1 * GL;
    constexpr int T = desc_tiles(L);
    constexpr int HALVES = T <= 16 ? 2 : 1, LANES_T = 32 / HALVES;
    constexpr int TPL = (T + LANES_T - 1) / LANES_T;                     // tiles per lane (1, or 2 from l_max = 10 on)
    constexpr int NB = (TPL * NP * 4 <= 64) ? NP : 64 / (4 * TPL);      // n handled per pass (at most 64 accumulators)
    constexpr int NPASS = (NP + NB - 1) / NB;
    constexpr int CPAIRS = NCHP / 2, ROUNDS = (CPAIRS + 31) / 32;       // lanes take pairs of adjacent n
    extern __shared__ __align__(16) float smem[];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, warps = blockDim.x >> 5;
    const bool o_cross = PLAIN || p.crossover, o_emit = !PLAIN && p.emit_coeff;
    const float* const o_cbar = PLAIN ? nullptr : p.c_bar;
    const float* const o_sites = PLAIN ? nullptr : p.sites;
    const float2* const o_pw = PLAIN ? nullptr : p.pair_w;
    const float o_w0 = PLAIN ? 1.f : p.w0;
    const int S = p.S, NMAX = p.n_max, F = p.F;
    const DescLayout lay = make_desc_layout(S, NP, L, warps, TS ? p.n_intervals * NCHP * 6 : 0);

    if (TS) {
        const float4* src = reinterpret_cast<const float4*>(p.table_ln);
        float4* dst = reinterpret_cast<float4*>(smem);
        const int n4 = p.n_intervals * NCHP * 6 / 4;
        for (int e = threadIdx.x; e < n4; e += blockDim.x) dst[e] = __ldg(src + e);
        __syncthreads();
    }
    // the table is this handle's own; everything below reads what the kernels before this one wrote
    grid_dependency_wait();
    // a failed neighbour build: write nothing
    if (p.counters->n_pairs > p.pair_capacity) return;

    float* const wbase = smem + lay.warp0 + wid * lay.per_warp;
    float* const c_t = wbase + lay.c;                                               // [LM][4 RC], chunks rotated by row / 4
    const int RC = desc_c_chunks(S, NP), rc_mask = RC - 1;
    auto c_chunk = [&](int r, int k) { return r * RC + ((k + (r >> 2)) & rc_mask); };        // 16-byte chunk k of row r
    auto c_word = [&](int r, int col) { return 4 * c_chunk(r, col >> 2) + (col & 3); };
    float4* const sS4 = reinterpret_cast<float4*>(wbase + lay.sS);                  // [chunk][SROW / 4] tiles of four m
    float* const sG = wbase + lay.sG;                                               // [chunk][L1][GL]
    float4* const ring_d = reinterpret_cast<float4*>(wbase + lay.ring);             // [chunk] dx, dy, dz, r
    int4* const ring_i = reinterpret_cast<int4*>(wbase + lay.ring + 4 * kDescChunk);// [chunk] interval, t, species, weight
    int* const ring_q = reinterpret_cast<int*>(wbase + lay.ring + 4 * kDescChunk);  // TS: [chunk] interval | species << 16, and t in ring_d.w
    float* const slab = wbase + lay.sS;
    const float4* const tab = TS ? reinterpret_cast<const float4*>(smem) : reinterpret_cast<const float4*>(p.table_ln);

    // the tiles of this lane: l, tile index, first row (l^2 + 4 j) and number of valid rows
    const int half = HALVES == 2 ? lane >> 4 : 0;
    int t_l[TPL], t_idx[TPL], t_lm0[TPL], t_kv[TPL];
#pragma unroll
    for (int tp = 0; tp < TPL; ++tp) {
        int t = tp * LANES_T + (lane & (LANES_T - 1)), l = 0;
        t_idx[tp] = t < T ? t : 0;
        if (t >= T) { t_l[tp] = 0; t_lm0[tp] = 0; t_kv[tp] = 0; continue; }
        while (t >= (2 * l + 4) / 4) { t -= (2 * l + 4) / 4; ++l; }
        t_l[tp] = l; t_lm0[tp] = l * l + 4 * t; t_kv[tp] = min(4, 2 * l + 1 - 4 * t);
    }
    // where this lane puts the radial factors it evaluates: the channel pair cp = l NP/2 + n/2 of round rr goes to
    // words l GL + n, l GL + n + 1
    int g_word[ROUNDS];
#pragma unroll
    for (int rr = 0; rr < ROUNDS; ++rr) {
        const int cp = rr * 32 + lane, l = cp / (NP / 2), n = 2 * (cp - l * (NP / 2));
        g_word[rr] = l * GL + 4 * ((n >> 2) ^ desc_g_swap(NP, l)) + (n & 3);
    }
    const bool periodic = p.geom.pbc[0] | p.geom.pbc[1] | p.geom.pbc[2];
    const long long n_work = o_cbar ? 1 : p.n_centers;

    // Centres are dealt out to the warps of the grid in turn (neighbouring warps take neighbouring centres).
    constexpr int PPL = kDescGroup / 32;                                 // pairs per lane and group
    struct Head { float xi, yi, zi; int zsp; long long pair_base; int k_pairs; };
    struct Raw { unsigned long long key[PPL]; float wgt[PPL]; int spj[PPL]; float px[PPL], py[PPL], pz[PPL]; };
    auto load_head = [&](long long c_idx) {
        Head h;
        const int ci = o_sites ? -1 : (p.centers ? p.centers[c_idx] : (int)c_idx);
        const float* pc = o_sites ? o_sites + 3 * c_idx : p.pos + 3 * (long long)ci;
        h.xi = pc[0]; h.yi = pc[1]; h.zi = pc[2];
        h.zsp = o_sites ? 0 : p.species_idx[ci];
        h.pair_base = p.pair_start[c_idx];
        h.k_pairs = o_cbar ? 0 : p.pair_count[c_idx];
        return h;
    };
    auto load_keys = [&](const Head& h, int g0, Raw& r) {
#pragma unroll
        for (int b = 0; b < PPL; ++b) {
            const int e = g0 + 32 * b + lane;
            r.key[b] = e < h.k_pairs ? p.pair_key[h.pair_base + e] : 0ull;
            r.wgt[b] = (o_pw && e < h.k_pairs) ? o_pw[h.pair_base + e].x : 1.f;
        }
    };
    auto load_atoms = [&](const Head& h, int g0, Raw& r) {
#pragma unroll
        for (int b = 0; b < PPL; ++b) {
            const int e = g0 + 32 * b + lane;
            r.spj[b] = -1; r.px[b] = r.py[b] = r.pz[b] = 0.f;
            if (e < h.k_pairs) {
                const int j = key_atom(r.key[b]);
                r.spj[b] = S == 1 ? 0 : p.species_idx[j];
                r.px[b] = p.pos[3 * (long long)j]; r.py[b] = p.pos[3 * (long long)j + 1]; r.pz[b] = p.pos[3 * (long long)j + 2];
            }
        }
    };
    // Full rounds give every warp of the grid one centre, CTA by CTA; the centres of the last, partial round are
    // dealt out across the CTAs first, so that every SM gets its share of them instead of a few SMs a full round
    const long long w_stride = (long long)gridDim.x * warps, full_rounds = n_work / w_stride;
    for (long long round = 0; round <= full_rounds; ++round) {
        const long long c_idx = round * w_stride + (round < full_rounds ? (long long)blockIdx.x * warps + wid
                                                                         : (long long)wid * gridDim.x + blockIdx.x);
        if (c_idx >= n_work) break;
        const Head hd = load_head(c_idx);
        Raw raw;
        const float xi = hd.xi, yi = hd.yi, zi = hd.zi;
        const int zi_species = hd.zsp, k_pairs = hd.k_pairs;

        for (int e = lane; e < LM * RC; e += 32) reinterpret_cast<float4*>(c_t)[e] = make_float4(0.f, 0.f, 0.f, 0.f);
        __syncwarp();

        for (int g0 = 0; g0 < k_pairs; g0 += kDescGroup) {
            // ---- geometry of up to 64 pairs, two per lane ----
            const int kg = min(kDescGroup, k_pairs - g0);
            load_keys(hd, g0, raw);
            load_atoms(hd, g0, raw);
            int sp[PPL], pos_sorted[PPL];
            float4 dd[PPL];
            int2 qt[PPL];                                                    // interval, offset bits
            float ww[PPL];
#pragma unroll
            for (int b = 0; b < PPL; ++b) {
                sp[b] = raw.spj[b];
                ww[b] = raw.wgt[b];
                dd[b] = make_float4(0.f, 0.f, 0.f, 0.f);
                qt[b] = make_int2(0, 0);
                pos_sorted[b] = -1;
                if (sp[b] >= 0) {
                    double dx = (double)raw.px[b] - (double)xi;
                    double dy = (double)raw.py[b] - (double)yi;
                    double dz = (double)raw.pz[b] - (double)zi;
                    if (periodic) {
                        int sh[3];
                        key_shift(raw.key[b], sh);
                        dx += sh[0] * p.geom.cell[0] + sh[1] * p.geom.cell[3] + sh[2] * p.geom.cell[6];
                        dy += sh[0] * p.geom.cell[1] + sh[1] * p.geom.cell[4] + sh[2] * p.geom.cell[7];
                        dz += sh[0] * p.geom.cell[2] + sh[1] * p.geom.cell[5] + sh[2] * p.geom.cell[8];
                    }
                    const double r = sqrt(dx * dx + dy * dy + dz * dz);
                    // interval and offset in the radial table, in fp64 so that the offset keeps its digits
                    const double u = r * p.inv_h;
                    const int qi = min((int)u, p.n_intervals - 1);
                    dd[b] = make_float4((float)dx, (float)dy, (float)dz, (float)r);
                    qt[b] = make_int2(qi, __float_as_int((float)(u - qi)));
                }
            }
            // position of every pair in species order (stable): ballots, no memory traffic
            {
                int base = 0;
                for (int s = 0; s < S; ++s)
#pragma unroll
                    for (int b = 0; b < PPL; ++b) {
                        const unsigned m = __ballot_sync(0xffffffffu, sp[b] == s);
                        if (sp[b] == s) pos_sorted[b] = base + __popc(m & ((1u << lane) - 1));
                        base += __popc(m);
                    }
            }

#pragma unroll 1
            for (int ip = 0; ip < NPASS; ++ip) {
                const int n0 = ip * NB;
                float2 acc[TPL][4][NB / 2];
#pragma unroll
                for (int tp = 0; tp < TPL; ++tp)
#pragma unroll
                    for (int k = 0; k < 4; ++k)
#pragma unroll
                        for (int n = 0; n < NB / 2; ++n) acc[tp][k][n] = make_float2(0.f, 0.f);
                int cur = -1;
                const bool single = k_pairs <= kDescGroup;            // one group: every (row, species) is written once

                // sums of species s (columns n0 .. n0 + NB - 1) are added to the centre's tile; the two half-warps add up first
                auto flush = [&](int s) {
#pragma unroll
                    for (int tp = 0; tp < TPL; ++tp)
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            float v[NB];
#pragma unroll
                            for (int n = 0; n < NB; ++n) {
                                v[n] = (n & 1) ? acc[tp][k][n / 2].y : acc[tp][k][n / 2].x;
                                if (HALVES == 2) v[n] += __shfl_xor_sync(0xffffffffu, v[n], 16);
                            }
#pragma unroll
                            for (int n = 0; n < NB / 2; ++n) acc[tp][k][n] = make_float2(0.f, 0.f);
                            if (k < t_kv[tp] && (HALVES == 1 || (k >> 1) == half)) {
                                float4* const c4w = reinterpret_cast<float4*>(c_t);
                                const int r = t_lm0[tp] + k, k0 = (s * NP + n0) / 4;
#pragma unroll
                                for (int n4 = 0; n4 < NB / 4; ++n4)
                                    if (NPASS == 1 || n0 + 4 * n4 < NP) {
                                        float4 o = make_float4(v[4 * n4], v[4 * n4 + 1], v[4 * n4 + 2], v[4 * n4 + 3]);
                                        float4* dst = c4w + c_chunk(r, k0 + n4);
                                        if (!single) {
                                            const float4 old = *dst;
                                            o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                                        }
                                        *dst = o;
                                    }
                            }
                        }
                };

                for (int c0 = 0; c0 < kg; c0 += kDescChunk) {
                    const int n_stage = min(kDescChunk, kg - c0);
                    // the pairs at sorted positions c0 .. c0 + 15 go to the staging slots
#pragma unroll
                    for (int b = 0; b < PPL; ++b)
                        if ((unsigned)(pos_sorted[b] - c0) < (unsigned)kDescChunk) {
                            if (TS) {
                                ring_d[pos_sorted[b] - c0] = make_float4(dd[b].x, dd[b].y, dd[b].z, __int_as_float(qt[b].y));
                                ring_q[pos_sorted[b] - c0] = qt[b].x | (sp[b] << 16);
                            } else {
                                ring_d[pos_sorted[b] - c0] = dd[b];
                                ring_i[pos_sorted[b] - c0] = make_int4(qt[b].x, qt[b].y, sp[b], __float_as_int(ww[b]));
                            }
                        }
                    __syncwarp();
                    // solid harmonics: a lane per pair
                    if (lane < n_stage) {
                        const float4 d = ring_d[lane];
                        harmonics_tiles<L>(d.x, d.y, d.z, TS ? fmaf(d.x, d.x, fmaf(d.y, d.y, d.z * d.z)) : d.w * d.w, sS4 + lane * (SROW / 4));
                    }
                    // radial factors: lanes on the channels, pairs in turn
#pragma unroll 4
                    for (int pr = 0; pr < n_stage; ++pr) {
                        int4 gi;
                        if (TS) { gi = make_int4(ring_q[pr] & 0xffff, __float_as_int(ring_d[pr].w), 0, 0); }
                        else gi = ring_i[pr];
                        const float t = __int_as_float(gi.y);
                        const float2 tt = make_float2(t, t);
                        const float4* row = tab + (size_t)gi.x * (NCHP * 6 / 4);
#pragma unroll
                        for (int rr = 0; rr < ROUNDS; ++rr) {
                            const int cp = rr * 32 + lane;
                            if (ROUNDS * 32 == CPAIRS || cp < CPAIRS) {
                                // coefficients of t^0 .. t^5 of two adjacent n, interleaved: (c0, c0', c1, c1'), (c2, c2', c3, c3'), (c4, c4', c5, c5')
                                const float4 A = TS ? row[cp * 3] : __ldg(row + cp * 3);
                                const float4 B = TS ? row[cp * 3 + 1] : __ldg(row + cp * 3 + 1);
                                const float4 C = TS ? row[cp * 3 + 2] : __ldg(row + cp * 3 + 2);
                                float2 v = __ffma2_rn(make_float2(C.z, C.w), tt, make_float2(C.x, C.y));
                                v = __ffma2_rn(v, tt, make_float2(B.z, B.w));
                                v = __ffma2_rn(v, tt, make_float2(B.x, B.y));
                                v = __ffma2_rn(v, tt, make_float2(A.z, A.w));
                                v = __ffma2_rn(v, tt, make_float2(A.x, A.y));
                                if (!PLAIN) { const float wgt = __int_as_float(gi.w); v.x *= wgt; v.y *= wgt; }
                                *reinterpret_cast<float2*>(sG + pr * GROW + g_word[rr]) = v;
                            }
                        }
                    }
                    __syncwarp();
                    const int tag = lane < n_stage ? (TS ? ring_q[lane] >> 16 : ring_i[lane].z) : -1;
                    for (int s = 0; s < S; ++s) {
                        const unsigned mask = __ballot_sync(0xffffffffu, tag == s);
                        if (!mask) continue;
                        const int a = __ffs(mask) - 1, b = a + __popc(mask);       // contiguous: staged in species order
                        if (s != cur) {
                            if (cur >= 0) flush(cur);
                            cur = s;
                        }
#pragma unroll 2
                        for (int q = a + half; q < b; q += HALVES) {
                            const float4* sp4 = sS4 + q * (SROW / 4);
                            const float4* gp = reinterpret_cast<const float4*>(sG + q * GROW + n0);
#pragma unroll
                            for (int tp = 0; tp < TPL; ++tp) {
                                const float4 h4 = sp4[t_idx[tp]];
                                const float2 h[4] = {make_float2(h4.x, h4.x), make_float2(h4.y, h4.y), make_float2(h4.z, h4.z),
                                                     make_float2(h4.w, h4.w)};
#pragma unroll
                                for (int n4 = 0; n4 < NB / 4; ++n4) {
                                    if (NPASS > 1 && n0 + 4 * n4 >= NP) break;
                                    const float4 g = gp[t_l[tp] * (GL / 4) + (n4 ^ desc_g_swap(NP, t_l[tp]))];
#pragma unroll
                                    for (int k = 0; k < 4; ++k) {
                                        acc[tp][k][2 * n4] = __ffma2_rn(h[k], make_float2(g.x, g.y), acc[tp][k][2 * n4]);
                                        acc[tp][k][2 * n4 + 1] = __ffma2_rn(h[k], make_float2(g.z, g.w), acc[tp][k][2 * n4 + 1]);
                                    }
                                }
                            }
                        }
                    }
                    __syncwarp();
                }
                if (cur >= 0) flush(cur);
                __syncwarp();
            }
        }

        // on-site term: the centre's own Gaussian, l = 0 only (second term of Eq. 13)
        if (!o_cbar && !o_sites && lane < NMAX) c_t[c_word(0, zi_species * NP + lane)] += o_w0 * __ldg(p.self_term + lane);
        if (o_cbar) {
            // given mean coefficients (inner average) take the place of the centre's own: index (mu n_max + n) LM + lm
            for (int e = lane; e < S * NMAX * LM; e += 32) {
                const int row = e / LM, lm = e - row * LM, mu = row / NMAX, n = row - mu * NMAX;
                c_t[c_word(lm, mu * NP + n)] = __ldg(o_cbar + e);
            }
        }
        __syncwarp();
        if (o_emit) {
            // coefficient mode: the tile itself is the result, index (mu n_max + n) (l_max+1)^2 + l^2 + l + m
            float* crow = p.out_desc + (size_t)c_idx * (S * NMAX * LM);
            for (int e = lane; e < S * NMAX * LM; e += 32) {
                const int row = e / LM, lm = e - row * LM, mu = row / NMAX, n = row - mu * NMAX;
                crow[e] = c_t[c_word(lm, mu * NP + n)];
            }
            __syncwarp();
            continue;
        }

        // ---- power spectrum (Eq. 4): per l the Gram matrix of the tile's rows over (species, n) ----
        float* const desc_row = p.out_desc + (o_cbar ? (size_t)0 : (size_t)c_idx * F);
        const bool staged = F <= lay.slab_words;
        float* const dst = staged ? slab : desc_row;
        // Lanes take blocks of 4 x 4 (species, n) pairs (ta <= tb in units of four columns); a block's place in the
        // feature row does not depend on l, so it is decoded once, and the lanes then walk down the l (with few
        // blocks, several l side by side: group g of the lanes takes l = l_max - g, l_max - g - G, ...).
        constexpr int TB = NP / 4;                                   // 4-wide column tiles per species
        const int TA = S * TB;
        const int NTP = o_cross ? TA * (TA + 1) / 2 : S * (TB * (TB + 1) / 2);
        const int G = NTP <= 16 ? 32 / NTP : 1;                      // l's side by side
        const int TRI = (NMAX * (NMAX + 1) / 2) * L1, SQ = NMAX * NMAX * L1;
        const float4* const c4 = reinterpret_cast<const float4*>(c_t);
        for (int tp0 = 0; tp0 < NTP; tp0 += 32) {
            const int grp = G > 1 ? lane / NTP : 0;
            int rem = G > 1 ? lane - grp * NTP : tp0 + lane;
            const bool active = grp < G && rem < NTP;
            if (!active) rem = 0;
            int ta = 0, tb = 0;
            if (o_cross) {
                while (rem >= TA - ta) { rem -= TA - ta; ++ta; }
                tb = ta + rem;
            } else {
                const int sb = rem / (TB * (TB + 1) / 2);
                rem -= sb * (TB * (TB + 1) / 2);
                while (rem >= TB - ta) { rem -= TB - ta; ++ta; }
                tb = sb * TB + ta + rem;
                ta += sb * TB;
            }
            // row i of the block starts at feature offset rowoff[i] (+ j (l_max+1) + l); bit 4 i + j of `valid` says
            // whether (i, j) is a feature at all (n below n_max, and n' >= n inside a diagonal species block)
            const int mu = (4 * ta) / NP, nu = (4 * tb) / NP, na = 4 * ta - mu * NP, nb = 4 * tb - nu * NP;
            int rowoff[4];
            unsigned valid = 0;
            {
                const int before = o_cross ? mu * S - mu * (mu - 1) / 2 + (nu - mu) : mu, diag = o_cross ? mu + (nu > mu ? 1 : 0) : mu;
                const int base = diag * TRI + (before - diag) * SQ;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int n1 = na + i;
                    rowoff[i] = base + (mu < nu ? n1 * NMAX + nb : n1 * NMAX - n1 * (n1 - 1) / 2 - n1 + nb) * L1;
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (active && n1 < NMAX && nb + j < NMAX && (mu < nu || n1 <= nb + j)) valid |= 1u << (4 * i + j);
                }
            }
            for (int l0 = L; l0 >= 0; l0 -= G) {
                const int l = l0 - grp;                                // this lane's l (may fall below zero in the last trip)
                const int steps = (active && l >= 0) ? 2 * l + 1 : 0;
                float2 g[4][2];
#pragma unroll
                for (int i = 0; i < 4; ++i) g[i][0] = g[i][1] = make_float2(0.f, 0.f);
                const int r0 = l >= 0 ? l * l : 0;
                for (int m = 0; m < steps; ++m) {
                    const float4 A = c4[c_chunk(r0 + m, ta)];
                    const float4 B = c4[c_chunk(r0 + m, tb)];
                    const float2 b01 = make_float2(B.x, B.y), b23 = make_float2(B.z, B.w);
                    const float av[4] = {A.x, A.y, A.z, A.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float2 aa = make_float2(av[i], av[i]);
                        g[i][0] = __ffma2_rn(aa, b01, g[i][0]);
                        g[i][1] = __ffma2_rn(aa, b23, g[i][1]);
                    }
                }
                if (steps) {
                    const float kl = __ldg(p.kl + l);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float* o = dst + rowoff[i] + l;
                        if (valid & (1u << (4 * i))) o[0] = kl * g[i][0].x;
                        if (valid & (2u << (4 * i))) o[L1] = kl * g[i][0].y;
                        if (valid & (4u << (4 * i))) o[2 * L1] = kl * g[i][1].x;
                        if (valid & (8u << (4 * i))) o[3 * L1] = kl * g[i][1].y;
                    }
                }
            }
        }
        __syncwarp();
        if (staged) {
            for (int e = lane; e < F; e += 32) desc_row[e] = slab[e];
            __syncwarp();
        }
    }
}

}  // namespace soap
