// The fused per-centre derivative kernel: one CTA owns one centre atom and produces its
// descriptor row (Eq. 4) and all of its Jacobian rows (Eq. 5).  (The descriptor-only
// build has a kernel of its own, desc_kernel.cuh.)  Nothing per pair ever goes to HBM: radial factors, solid
// harmonics and the precontracted U/V live in shared memory; the expansion
// coefficients c^mu_nlm of the centre stay in shared memory for the CTA's life.
//
// Per pair (displacement d = r_j + T - r_i, species Z of j):
//   c^Z_nlm        += G_nl(|d|) S_lm(d)                               (Eq. 13 / 18)
//   grad_j c^Z_nlm  = G_nl grad S_lm + Ghat_nl d S_lm,  Ghat = G'/|d|  (Eq. 14 / 23)
// with S_lm = r^l Y_lm the real solid harmonic and G_nl, G'_nl read from the
// degree-5 tables.
//   Staging (whole CTA, a chunk of up to 32 pairs): radial factors with a warp per
//   pair and lanes on channels; solid harmonics with lanes on pairs and warps on
//   the columns m of the recursion, so that control flow is uniform.
//   Pass 1 accumulates c and D = sum_j grad_j c with thread-owned elements; the
//   centre's own Jacobian row is minus the sum over its neighbours (translation
//   invariance, text below Eq. 5), which is a contraction of D with c.
//   Pass 2 gives every pair to one warp: it forms U^nu_{n'l} = K_l sum_m S_lm
//   c^nu_{n'lm} and V likewise with grad S, after which every output element of
//   Eq. 5 is two fused multiply-adds per term, and streams the row out with lanes
//   on consecutive features.
// l_max and n_max are template parameters (n_max = 0 means "read it at run
// time") so that loops unroll and the store addresses become immediates.
#pragma once
#include <type_traits>

#include "soap_device.cuh"

constexpr int kTriUnroll = 2;          // sweeps of a same-species block in flight per warp
constexpr int kMinCtas = 3;            // resident CTAs per SM the kernel is compiled for

namespace soap {

// Universal small tables for the harmonic recursion (l_max <= 12), read with
// warp-uniform indices, hence constant memory.  Each translation unit that
// includes this file gets its own copy, filled in at load time.
__device__ __constant__ float2 kc_norm[91] = {0};    // [(l,m)] a_lm = sqrt((2l+1)/4pi (l-m)!/(l+m)!) (sqrt2 for m > 0), (l+m) a_lm
__device__ __constant__ float4 kc_step[91] = {0};    // [(l,m)] coefficients that advance columns m and m+1 from l to l+1
__device__ __constant__ float kc_dfact[16] = {0};    // [m] (2m-1)!!

// Degree-5 table lookup: value and derivative with respect to the interval coordinate t.
__device__ __forceinline__ void radial_lookup(const float* __restrict__ table, int qi, int n_ch, int ch, float t,
                                              float& v, float& dv) {
    // 32-bit index arithmetic: the table has at most 4096 x 208 x 6 floats
    const float2* cf = reinterpret_cast<const float2*>(table) + (unsigned)(qi * n_ch + ch) * 3u;
    const float2 a = __ldg(cf), b = __ldg(cf + 1), c = __ldg(cf + 2);
    v = c.y; dv = 0.f;
    dv = fmaf(dv, t, v); v = fmaf(v, t, c.x);
    dv = fmaf(dv, t, v); v = fmaf(v, t, b.y);
    dv = fmaf(dv, t, v); v = fmaf(v, t, b.x);
    dv = fmaf(dv, t, v); v = fmaf(v, t, a.y);
    dv = fmaf(dv, t, v); v = fmaf(v, t, a.x);
}

// Real solid harmonics of one pair per lane, one column m of
//   S_{l,+m} = a_lm Q_l^m Re (x+iy)^m,   S_{l,-m} = a_lm Q_l^m Im (x+iy)^m,
//   Q_l^m = r^(l-m) d^m P_l(t)/dt^m at t = z/r,
//   (l+1-m) Q_{l+1}^m = (2l+1) z Q_l^m - (l+m) r^2 Q_{l-1}^m,   Q_m^m = (2m-1)!!,
//   dQ_l^m/dx = -x Q_{l-1}^{m+1},  dQ_l^m/dy = -y Q_{l-1}^{m+1},  dQ_l^m/dz = (l+m) Q_{l-1}^m.
// Columns m and m+1 are advanced in lock step, so a step needs four registers; the rational
// coefficients of the recurrences come from constant memory (all lanes use the same (l, m)).
__device__ __forceinline__ void harmonics_column(int L, int m, float x, float y, float z, float r2, float4* __restrict__ out4) {
    float cm = 1.f, sm = 0.f, cp = 0.f, sp = 0.f;               // (x+iy)^m and (x+iy)^(m-1)
    for (int t = 0; t < m; ++t) {
        cp = cm; sp = sm;
        const float cn = x * cm - y * sm;
        sm = x * sm + y * cm;
        cm = cn;
    }
    float a1 = kc_dfact[m], a0 = 0.f;                           // Q_l^m, Q_{l-1}^m
    float b1 = 0.f, b0 = 0.f;                                   // Q_l^{m+1}, Q_{l-1}^{m+1}
    const float fm = (float)m;
    int t = m * (m + 1) / 2 + m;                                // index of (l, m), l = m
    for (int l = m; l <= L; ++l) {
        const float2 nr = kc_norm[t];
        const float aq = nr.x * a1;
        const int lm0 = l * l + l;
        const float qz = nr.y * a0;                             // a (l+m) Q_{l-1}^m  (a0 = 0 when l = m)
        const float qx = nr.x * b0;                             // a Q_{l-1}^{m+1}
        const float mq = fm * aq;
        const float xq = x * qx, yq = y * qx;
        out4[lm0 + m] = make_float4(aq * cm, mq * cp - xq * cm, -mq * sp - yq * cm, qz * cm);
        if (m) out4[lm0 - m] = make_float4(aq * sm, mq * sp - xq * sm, mq * cp - yq * sm, qz * sm);
        // advance both columns to l + 1
        const float4 st = kc_step[t];
        const float an = st.x * z * a1 - st.y * r2 * a0;
        a0 = a1; a1 = an;
        const float bn = (l == m) ? kc_dfact[m + 1] : st.z * z * b1 - st.w * r2 * b0;
        b0 = b1; b1 = bn;
        t += l + 1;
    }
}

// Bulk asynchronous copy shared -> global (the copy engine moves the bytes; one thread issues it).  Addresses and
// size must be multiples of 16 bytes.  Copies of a thread are grouped by bulk_commit(); bulk_wait_read() returns
// once the shared-memory source of all its groups has been read.
__device__ __forceinline__ void bulk_store(float* dst, const float* src_shared, unsigned bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 :: "l"(dst), "r"((unsigned)__cvta_generic_to_shared(src_shared)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

// KIND: 1 descriptor and Jacobian, 2 coefficients c^mu_nlm and their Jacobian, 3 Jacobian of the inner average
// (every atom a centre; given mean coefficients; one row per atom, no per-pair rows), 4 Jacobian of the outer average
// (every atom a centre; given the coefficients of all centres; one row per atom, no per-pair rows).
// PLAIN: the default configuration (every species pair, atom centres, no weighting, full rows, own
// coefficients); the options are then compile-time constants and their code drops out.
template <int KIND, int L, int NMAX_T, bool PLAIN>
__global__ void __launch_bounds__(kThreads, kMinCtas)
center_kernel(const CenterParams p) {
    static_assert(KIND >= 1 && KIND <= 4, "descriptor-only builds run desc_kernel");
    constexpr bool CC = KIND == 2;
    const bool o_compact = !PLAIN && p.compact, o_cross = PLAIN || p.crossover;
    const float* const o_cbar = PLAIN ? nullptr : p.c_bar;
    const float* const o_sites = PLAIN ? nullptr : p.sites;
    const float2* const o_pw = PLAIN ? nullptr : p.pair_w;
    const float o_w0 = PLAIN ? 1.f : p.w0;
    constexpr bool o_inner = KIND == 3, o_outer = KIND == 4;
    constexpr bool o_atom_rows = o_inner || o_outer;               // the result has one row per atom, at the atom's index
    const float o_scale = o_atom_rows ? p.own_scale : 1.f;
    constexpr int L1 = L + 1, LM = L1 * L1, LMP = LM | 1;      // odd row stride: no shared-memory bank conflicts
    constexpr int NMAX_BOUND = NMAX_T ? NMAX_T : 16;
    // pass-1 ownership: W_LM warps cover the lm index, SLOTS such groups split the n index
    constexpr int W_LM = (LM + 31) / 32;
    constexpr int SLOTS_FULL = kWarps / W_LM, SLOT_DIV = 2;
    constexpr int SLOTS = SLOTS_FULL / SLOT_DIV > 0 ? SLOTS_FULL / SLOT_DIV : 1;
    constexpr int NPT_RAW = (NMAX_BOUND + SLOTS - 1) / SLOTS;      // radial functions per thread ...
    constexpr int NPT = NPT_RAW < 8 ? NPT_RAW : 8;                // ... at most 8 at a time (register budget)
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int S = p.S, NMAX = NMAX_T ? NMAX_T : p.n_max, NCH = NMAX * L1, NE = NMAX * LM;
    const int CT = S * NMAX * LMP, P = p.P, F = p.F;
    const SmemLayout lay = make_layout(S, NMAX, L, P, true, o_pw != nullptr);
    float* c_t = smem + lay.c;                                             // [S][NMAX][LMP]
    float4* geo_d = reinterpret_cast<float4*>(smem + lay.geo);             // [GP] dx, dy, dz, r
    int4* geo_i = reinterpret_cast<int4*>(smem + lay.geo + 4 * kGeoPairs);   // [GP] interval, t bits, species|moving<<8, row word
    int* geo_j = reinterpret_cast<int*>(smem + lay.geo + 8 * kGeoPairs);     // [GP] neighbour atom
    float2* geo_w = reinterpret_cast<float2*>(smem + lay.geo + kGeoWords);   // [GP] (w, w'/d), only with a radial weighting
    float* D_t = smem + lay.D;                                             // [3][CT]    (pass 1 and the centre's row)
    float4* sSD4 = reinterpret_cast<float4*>(smem + lay.sSD);              // [P][LMP]   (S, dSx, dSy, dSz)
    float2* sG2 = reinterpret_cast<float2*>(smem + lay.sG);                // [P][NCH]   (G, Ghat)

    // ---- set-up that needs nothing from the kernels before this one (it may run while they finish) ----
    for (int e = tid; e < CT * 4; e += kThreads) {
        if (e < CT) c_t[e] = 0.f; else D_t[e - CT] = 0.f;
    }
    // zeros for the bulk copies of pass 2 (made visible to the copy engine; the barriers of pass 1 order them)
    const float* zero_buf = smem + lay.zero;
    for (int e = tid; e < kZeroWords; e += kThreads) smem[lay.zero + e] = 0.f;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");

    // same-species blocks: feature index -> (n1 L1 + l) | (n2 L1 + l) << 8, rows n1 of (NMAX - n1) L1 entries
    unsigned short* tri_dec = reinterpret_cast<unsigned short*>(smem + lay.tri);
    if (!CC)
        for (int e = tid; e < (NMAX * (NMAX + 1) / 2) * L1; e += kThreads) {
            int n1 = 0, r = e;
            while (r >= (NMAX - n1) * L1) { r -= (NMAX - n1) * L1; ++n1; }
            const int n2 = n1 + r / L1, l = r % L1;
            tri_dec[e] = (unsigned short)((n1 * L1 + l) | ((n2 * L1 + l) << 8));
        }
    // cross-species blocks (rows n1 of n_ch entries): feature index -> (n1 L1 + l) | (n2 L1 + l) << 8
    // (measured on the 1000-molecule cluster: 3 to 7 % faster than decoding every feature by arithmetic at n_max = 10;
    // up to n_max = 8 the lanes-on-columns path further down stays 1 to 6 % ahead)
    constexpr bool kCrossTable = KIND != 2 && NMAX_T > 8 && NMAX_T <= 12 && ((NMAX_BOUND * L1) & 3) != 0;
    unsigned short* x_dec = reinterpret_cast<unsigned short*>(smem + lay.xdec);
    if (kCrossTable && S > 1)
        for (int e = tid; e < NMAX * NCH; e += kThreads) {
            const int n1 = e / NCH, j = e - n1 * NCH;
            x_dec[e] = (unsigned short)((n1 * L1 + j % L1) | (j << 8));
        }

    // ---- from here on the neighbour data of this call is read ----
    grid_dependency_wait();
    const long long c_idx = p.order ? p.order[blockIdx.x] : blockIdx.x;
    // a failed neighbour build or an undersized output: write nothing
    if (p.counters->n_pairs > p.pair_capacity) return;
    if (p.row_ptr[p.n_centers] > p.row_capacity) {
        if (c_idx == 0 && tid == 0) atomicOr(&p.counters->status, kStatusRowCapacity);
        return;
    }
    const int ci = o_sites ? -1 : (p.centers ? p.centers[c_idx] : (int)c_idx);
    const float* pc = o_sites ? o_sites + 3 * c_idx : p.pos + 3 * (long long)ci;
    const float xi = pc[0], yi = pc[1], zi = pc[2];
    const int zi_species = o_sites ? 0 : p.species_idx[ci];
    const long long pair_base = p.pair_start[c_idx];
    const int k_pairs = p.pair_count[c_idx];
    const bool periodic = p.geom.pbc[0] | p.geom.pbc[1] | p.geom.pbc[2];
    // the pairs are taken in batches of geometry of equal size (a multiple of eight, at most kGeoPairs): 274 pairs are
    // 96 + 96 + 82, not 128 + 128 + 18
    const int geo_batches = (k_pairs + kGeoPairs - 1) / kGeoPairs;
    const int geo_batch = geo_batches > 1 ? min(kGeoPairs, (((k_pairs + geo_batches - 1) / geo_batches) + 7) & ~7) : kGeoPairs;

    // pass-1 ownership of this thread: one lm, and the radial functions slot, slot + SLOTS, ...
    const int own_slot = wid / W_LM, own_lm = (wid - own_slot * W_LM) * 32 + lane;
    const bool owner = own_slot < SLOTS && own_lm < LM;
    const int own_l = owner ? __ldg(p.l_of_lm + own_lm) : 0;

    // ---- geometry of up to kGeoPairs pairs, one thread each, stored grouped by the neighbour's
    //      species (stable, so images of one atom stay adjacent and in order); seg[s] .. seg[s+1]
    //      are the pairs of species s.  Returns whether any pair of the batch shares its row with
    //      another or is an image of the centre ----
    int* seg = reinterpret_cast<int*>(smem + lay.geo + 9 * kGeoPairs);       // [kMaxSpecies + 1]
    int* seg_warp = seg + kMaxSpecies + 1;                                   // [4 warps][kMaxSpecies]
    auto stage_geometry = [&](int g0, int gc) -> bool {
        int special = 0, sp = -1, rank = 0, rw = 0, j = 0;
        float4 dd = make_float4(0.f, 0.f, 0.f, 0.f);
        float2 wgt = make_float2(1.f, 0.f);
        int qi = 0;
        float tt = 0.f;
        if (tid < kGeoPairs) {
            if (tid < gc) {
                const unsigned long long key = p.pair_key[pair_base + g0 + tid];
                j = key_atom(key);
                double dx = (double)p.pos[3 * (long long)j] - (double)xi;
                double dy = (double)p.pos[3 * (long long)j + 1] - (double)yi;
                double dz = (double)p.pos[3 * (long long)j + 2] - (double)zi;
                if (periodic) {
                    int s[3];
                    key_shift(key, s);
                    dx += s[0] * p.geom.cell[0] + s[1] * p.geom.cell[3] + s[2] * p.geom.cell[6];
                    dy += s[0] * p.geom.cell[1] + s[1] * p.geom.cell[4] + s[2] * p.geom.cell[7];
                    dz += s[0] * p.geom.cell[2] + s[1] * p.geom.cell[5] + s[2] * p.geom.cell[8];
                }
                const double r = sqrt(dx * dx + dy * dy + dz * dz);
                dd = make_float4((float)dx, (float)dy, (float)dz, (float)r);
                rw = p.pair_row[pair_base + g0 + tid];
                if (o_pw) wgt = o_pw[pair_base + g0 + tid];
                special = rw & (kRowSelfImage | kRowContinuation);
                // interval and offset in the radial table, in fp64 so that the offset keeps its digits
                const double u = r * p.inv_h;
                qi = min((int)u, p.n_intervals - 1);
                tt = (float)(u - qi);
                sp = p.species_idx[j];
            }
            // stable partition by species: rank inside the warp, then offsets across warps
            for (int s = 0; s < S; ++s) {
                const unsigned m = __ballot_sync(0xffffffffu, sp == s);
                if (sp == s) rank = __popc(m & ((1u << lane) - 1));
                if (lane == 0) seg_warp[wid * kMaxSpecies + s] = __popc(m);
            }
        }
        const bool any_special = __syncthreads_or(special) != 0;
        if (tid < gc) {
            int at = rank;
            for (int s = 0; s < sp; ++s)
                for (int w = 0; w < kGeoPairs / 32; ++w) at += seg_warp[w * kMaxSpecies + s];
            for (int w = 0; w < wid; ++w) at += seg_warp[w * kMaxSpecies + sp];
            geo_d[at] = dd;
            geo_i[at] = make_int4(qi, __float_as_int(tt), sp | ((rw & kRowSelfImage) ? 0 : 256), rw);
            geo_j[at] = j;
            if (o_pw) geo_w[at] = wgt;
        }
        if (tid <= S) {
            int at = 0;
            for (int s = 0; s < tid; ++s)
                for (int w = 0; w < kGeoPairs / 32; ++w) at += seg_warp[w * kMaxSpecies + s];
            seg[tid] = at;
        }
        __syncthreads();
        return any_special;
    };

    // ---- radial factors and solid harmonics of the pairs g .. g + pc - 1 of the staged geometry ----
    auto stage_chunk = [&](int g, int pc) {
        for (int pr = wid; pr < pc; pr += kWarps) {
            const int4 gi = geo_i[g + pr];
            const float t = __int_as_float(gi.y);
            const float rinv_h = (float)p.inv_h / geo_d[g + pr].w;
            if (o_pw) {
                // radial weighting: G -> w G, Ghat -> w Ghat + (w'/d) G
                const float2 w = geo_w[g + pr];
                for (int ch = lane; ch < NCH; ch += 32) {
                    float v, dv;
                    radial_lookup(p.table, gi.x, NCH, ch, t, v, dv);
                    sG2[pr * NCH + ch] = make_float2(v * w.x, fmaf(dv * rinv_h, w.x, v * w.y));
                }
                continue;
            }
            for (int ch = lane; ch < NCH; ch += 32) {
                float v, dv;
                radial_lookup(p.table, gi.x, NCH, ch, t, v, dv);
                sG2[pr * NCH + ch] = make_float2(v, dv * rinv_h);
            }
        }
        if (P >= 32) {
            // a warp per column: m is the same for all its lanes, so the recursion's coefficients are uniform reads
            if (lane < pc) {
                const float4 d = geo_d[g + lane];
                for (int m = wid; m <= L; m += kWarps)
                    harmonics_column(L, m, d.x, d.y, d.z, d.w * d.w, sSD4 + lane * LMP);
            }
        } else {
            // the staging area holds 16 pairs or fewer: the lanes of a warp take several columns side by side (more of
            // them for a short chunk), so that the recursion runs over fewer trips
            // (the span follows the chunk only from l_max = 9 on: below, the extra code cost the headline build 0.5 %)
            const int span = L >= 9 ? (pc > 8 ? 16 : pc > 4 ? 8 : 4) : P, cols = 32 / span, pr = lane & (span - 1), cg = lane / span;
            if (pr < pc) {
                const float4 d = geo_d[g + pr];
                for (int m = wid * cols + cg; m <= L; m += kWarps * cols)
                    harmonics_column(L, m, d.x, d.y, d.z, d.w * d.w, sSD4 + pr * LMP);
            }
        }
    };

    // =========================== pass 1: c (and D) ===========================
    // A thread owns c[s][n][own_lm] (and the three D tiles) for its n and keeps the sums of the
    // species it is working on in registers; pairs arrive grouped by species, so the sums go to
    // shared memory once per species and batch.
    bool special = false;
    for (int n0 = 0; n0 < NMAX; n0 += SLOTS * NPT) {             // one trip unless n_max > 8 SLOTS
        for (int g0 = 0; g0 < k_pairs; g0 += geo_batch) {
            const int gc = min(geo_batch, k_pairs - g0);
            __syncthreads();
            special = stage_geometry(g0, gc);
            float ac[NPT], ax[NPT], ay[NPT], az[NPT];
            // inner average: q = sum over the neighbour centres i of grad_a c(i), the gradient of THEIR coefficients with
            // respect to this atom a.  Centre i sees a at -d, and [G grad S + Ghat d S](-d) = (-1)^(l+1) [..](d), so q
            // is built from the very terms that go into D; it belongs to the block of this atom's species
            float qx[NPT], qy[NPT], qz[NPT];
            const float q_sign = (own_l & 1) ? 1.f : -1.f;
#pragma unroll
            for (int k = 0; k < NPT; ++k) ac[k] = ax[k] = ay[k] = az[k] = qx[k] = qy[k] = qz[k] = 0.f;
            int cur = -1;
            auto flush = [&]() {
                if (cur < 0 || !owner) return;
#pragma unroll
                for (int k = 0; k < NPT; ++k) {
                    const int n = n0 + own_slot + k * SLOTS;
                    if (n < NMAX) {
                        const int e = (cur * NMAX + n) * LMP + own_lm;
                        c_t[e] += ac[k];
                        D_t[e] += ax[k]; D_t[CT + e] += ay[k]; D_t[2 * CT + e] += az[k];
                    }
                    ac[k] = ax[k] = ay[k] = az[k] = 0.f;
                }
            };
            for (int q0 = 0; q0 < gc; q0 += P) {
                const int pc = min(P, gc - q0);
                stage_chunk(q0, pc);
                __syncthreads();
                if (owner) {
                    for (int s = 0; s < S; ++s) {
                        const int a = max(seg[s], q0), b = min(seg[s + 1], q0 + pc);
                        if (a >= b) continue;
                        if (s != cur) { flush(); cur = s; }
                        for (int g = a; g < b; ++g) {
                            const int pr = g - q0;
                            {
                                const float4 h = sSD4[pr * LMP + own_lm];
                                const float4 d = geo_d[g];
                                // an image of the centre does not move relative to it: no contribution to D
                                // (only a batch with images or shared rows can hold one)
                                const float mv = (!special || (geo_i[g].z & 256)) ? 1.f : 0.f;
                                float hy = h.y, hz = h.z, hw = h.w, tx = h.x * d.x, ty = h.x * d.y, tz = h.x * d.z;
                                if (special) { hy *= mv; hz *= mv; hw *= mv; tx *= mv; ty *= mv; tz *= mv; }
                                const float2* gp = sG2 + pr * NCH + (n0 + own_slot) * L1 + own_l;
#pragma unroll
                                for (int k = 0; k < NPT; ++k)
                                    if (n0 + own_slot + k * SLOTS < NMAX) {
                                        const float2 gg = gp[k * SLOTS * L1];
                                        ac[k] = fmaf(gg.x, h.x, ac[k]);
                                        ax[k] = fmaf(gg.x, hy, fmaf(gg.y, tx, ax[k]));
                                        ay[k] = fmaf(gg.x, hz, fmaf(gg.y, ty, ay[k]));
                                        az[k] = fmaf(gg.x, hw, fmaf(gg.y, tz, az[k]));
                                        if (o_inner) {
                                            qx[k] = fmaf(q_sign, fmaf(gg.x, hy, gg.y * tx), qx[k]);
                                            qy[k] = fmaf(q_sign, fmaf(gg.x, hz, gg.y * ty), qy[k]);
                                            qz[k] = fmaf(q_sign, fmaf(gg.x, hw, gg.y * tz), qz[k]);
                                        }
                                    }
                            }
                        }
                    }
                }
                __syncthreads();
            }
            flush();
            if (o_inner && owner) {
                // D - q in the block of this atom's species: minus the sum over ALL centres of grad_a c, the centre itself included
#pragma unroll
                for (int k = 0; k < NPT; ++k) {
                    const int n = n0 + own_slot + k * SLOTS;
                    if (n < NMAX) {
                        const int e = (zi_species * NMAX + n) * LMP + own_lm;
                        D_t[e] -= qx[k]; D_t[CT + e] -= qy[k]; D_t[2 * CT + e] -= qz[k];
                    }
                }
            }
        }
    }
    __syncthreads();
    // on-site term: the centre's own Gaussian, l = 0 only (second term of Eq. 13)
    if (tid < NMAX && !o_cbar && !o_sites) c_t[(zi_species * NMAX + tid) * LMP] += o_w0 * __ldg(p.self_term + tid);
    __syncthreads();
    const int W = S * NE;                                                  // coefficients per centre
    const int RW = CC ? W : (o_compact ? p.Fc : F);                        // width of an output row
    if (o_cbar) {
        // inner average: the mean coefficients (on-site terms included) take the place of the centre's own
        for (int e = tid; e < W; e += kThreads) {
            const int row = e / LM;
            c_t[row * LMP + (e - row * LM)] = __ldg(o_cbar + e);
        }
        __syncthreads();
    }
    if (CC) {
        // coefficient mode: the tile itself is the result, index (mu n_max + n) (l_max+1)^2 + l^2 + l + m
        float* crow = p.out_desc + (size_t)c_idx * W;
        for (int e = tid; e < W; e += kThreads) {
            const int row = e / LM;
            crow[e] = c_t[row * LMP + (e - row * LM)];
        }
    }

    // ============ power spectrum (Eq. 4) and the centre's own row ============
    // Threads walk the features l-major so that the lanes of a warp share the trip count 2l+1; the
    // centre's row is minus the sum over its neighbours: -K_l sum_m (D^mu c^nu + c^mu D^nu).  Results
    // pass through the (now idle) staging area in slabs, so that global memory is written in
    // feature order, whole sectors at a time.
    const long long row_base = p.row_ptr[c_idx];
    const bool has_own = !o_sites;                   // a centre that is no atom has no row of its own
    if (CC) {
        // the centre's own row: minus the sum over the atoms that move relative to it
        if (has_own) {
            float* own = p.out_jac + (size_t)(row_base + p.self_row[c_idx]) * 3 * W;
            for (int e = tid; e < 3 * W; e += kThreads) {
                const int k = e / W, r = e - k * W, row = r / LM;
                own[e] = -D_t[k * CT + row * LMP + (r - row * LM)];
            }
            if (tid == 0) p.row_atom[row_base + p.self_row[c_idx]] = ci;
        }
    } else {
        // with given mean coefficients every centre would write the same descriptor: the first one does
        const bool write_desc = !o_cbar || c_idx == 0;
        float* desc_row = p.out_desc + (o_cbar ? (size_t)0 : (size_t)c_idx * F);
        // species-compact rows: the centre's own row keeps every block and lives in an array of its own;
        // its slot among the compact rows is zero-filled
        float* own = !has_own ? nullptr
                     : o_atom_rows ? p.out_jac + (size_t)ci * 3 * F            // row of atom a in the (atoms, 3, F) result
                     : o_compact ? p.out_center + (size_t)c_idx * 3 * F
                                 : p.out_jac + (size_t)(row_base + p.self_row[c_idx]) * 3 * F;
        if (has_own && o_compact) {
            float* slot = p.out_jac + (size_t)(row_base + p.self_row[c_idx]) * 3 * RW;
            for (int e = tid; e < 3 * RW; e += kThreads) slot[e] = 0.f;
        }
        float* slab = smem + lay.sSD;
        constexpr int NV = 4;                                               // values per feature: p and the three components of the centre's row
        const int NP = F / L1;                                              // (species pair, n, n') groups
        int gp = ((lay.total - lay.sSD) / NV) / L1;                         // groups per slab
        gp = gp < 1 ? 1 : (gp > NP ? NP : gp);
        const bool staged = (lay.total - lay.sSD) >= NV * L1;
        for (int q0 = 0; q0 < NP; q0 += gp) {
            const int nq = min(gp, NP - q0), nf = nq * L1, f0 = q0 * L1;
            for (int g = tid; g < nf; g += kThreads) {
                const int l = g / nq, fl = (g - l * nq) * L1 + l;             // feature index inside the slab
                const int pk = __ldg(p.feat_pack + f0 + fl);
                const int n1 = pk & 31, n2 = (pk >> 5) & 31, mu = (pk >> 10) & 15, nu = (pk >> 14) & 15;
                const int ia = (mu * NMAX + n1) * LMP + l * l, ib = (nu * NMAX + n2) * LMP + l * l;
                const float kl = __ldg(p.kl + l);
                float acc = 0.f, ax = 0.f, ay = 0.f, az = 0.f;
                for (int m = 0; m <= 2 * l; ++m) {
                    const float ca = c_t[ia + m], cb = c_t[ib + m];
                    acc = fmaf(ca, cb, acc);
                    ax = fmaf(D_t[ia + m], cb, fmaf(ca, D_t[ib + m], ax));
                    ay = fmaf(D_t[CT + ia + m], cb, fmaf(ca, D_t[CT + ib + m], ay));
                    az = fmaf(D_t[2 * CT + ia + m], cb, fmaf(ca, D_t[2 * CT + ib + m], az));
                }
                if (staged) {
                    slab[fl] = kl * acc;
                    const float ks = -kl * o_scale;
                    slab[nf + fl] = ks * ax; slab[2 * nf + fl] = ks * ay; slab[3 * nf + fl] = ks * az;
                } else {
                    if (write_desc) desc_row[f0 + fl] = kl * acc;
                    if (has_own) {
                        const float ks = -kl * o_scale;
                        own[f0 + fl] = ks * ax; own[(size_t)F + f0 + fl] = ks * ay; own[(size_t)2 * F + f0 + fl] = ks * az;
                    }
                }
            }
            if (staged) {
                __syncthreads();
                for (int e = tid; e < nf; e += kThreads) {
                    if (write_desc) desc_row[f0 + e] = slab[e];
                    if (has_own) {
                        own[f0 + e] = slab[nf + e];
                        own[(size_t)F + f0 + e] = slab[2 * nf + e];
                        own[(size_t)2 * F + f0 + e] = slab[3 * nf + e];
                    }
                }
                __syncthreads();
            }
        }
        if (has_own && !o_atom_rows && tid == 0) p.row_atom[row_base + p.self_row[c_idx]] = ci;
    }
    if (o_inner) return;             // the averaged row of this atom is complete: no per-pair rows
    __syncthreads();
    if constexpr (o_outer) {
        // Outer average with every atom a centre: d pbar / d r_a = (1/C) sum_i d p(i) / d r_a.  Besides its own row
        // (written above) atom a has a row under every centre i that sees it, and those are the atoms that a sees.
        // Centre i sees a at -d: S_lm(-d) = (-1)^l S_lm(d), grad S_lm(-d) = (-1)^(l+1) grad S_lm(d), and the
        // displacement in Ghat d S changes sign as well, so the row of a under i is the product rule of this very
        // pair with U, V contracted against c(i) instead of c(a), times (-1)^(l+1).  In rounds of one pair per warp:
        // a warp copies c(i) to shared memory and forms U, V; then the threads, each with features of its own, add
        // the pairs of the round in a fixed order (bit-repeatable).  Only the blocks that involve the species of a
        // are touched; a thread keeps its sums in registers over all rounds when they are at most kSlots features
        // per thread, else it adds to the row in global memory group by group, every round.
        constexpr int kSlots = 4;
        const int NI = S * NCH, SN = S * NMAX, Z = zi_species;
        const int TRI = (NMAX * (NMAX + 1) / 2) * L1, SQ = NMAX * NCH;
        const int NZ = TRI + (o_cross ? (S - 1) * SQ : 0);                     // features that involve species Z
        float4* sUV = reinterpret_cast<float4*>(smem + lay.wUV);              // [kWarps][nu][n'][l]
        float* c_copy = smem + lay.total + wid * CT;                          // [kWarps][S n_max][LMP], behind the usual layout
        float* const row = p.out_jac + (size_t)ci * 3 * F;
        // the x-th feature that involves Z: its place in the row and its operands, (radial index, U/V index) of one
        // term, or of both in the same-species block (gB >= 0)
        auto decode = [&](int x, int& f, int& gA, int& uA, int& gB, int& uB) {
            gB = -1; uB = 0;
            if (x < TRI) {
                // block (Z, Z): after the blocks (mu, nu >= mu) of every mu < Z
                f = o_cross ? Z * TRI + (Z * S - Z * (Z + 1) / 2) * SQ + x : Z * TRI + x;
                const unsigned dec = tri_dec[x];
                gA = dec & 255; gB = dec >> 8;
                uA = Z * NCH + gB; uB = Z * NCH + gA;
            } else {
                const int y = x - TRI, o = y / SQ, e = y - o * SQ;
                const int other = o < Z ? o : o + 1, mu = min(Z, other), nu = max(Z, other);
                f = mu * TRI + (mu * S - mu * (mu + 1) / 2) * SQ + TRI + (nu - mu - 1) * SQ + e;
                const int n1 = (int)__umulhi((unsigned)e, p.nch_magic);
                const int j = e - n1 * NCH, i1 = n1 * L1 + (j % L1);
                const bool first_term = mu == Z;                               // which factor belongs to atom a
                gA = first_term ? i1 : j;
                uA = other * NCH + (first_term ? j : i1);
            }
        };
        const int n_groups = (NZ + kSlots * kThreads - 1) / (kSlots * kThreads);
        const bool in_registers = n_groups == 1;
        int sf[kSlots], sgA[kSlots], suA[kSlots], sgB[kSlots], suB[kSlots];
        float ax[kSlots], ay[kSlots], az[kSlots];
#pragma unroll
        for (int k = 0; k < kSlots; ++k) {
            ax[k] = ay[k] = az[k] = 0.f;
            sf[k] = -1; sgA[k] = suA[k] = suB[k] = 0; sgB[k] = -1;
            if (in_registers && k * kThreads + tid < NZ) decode(k * kThreads + tid, sf[k], sgA[k], suA[k], sgB[k], suB[k]);
        }
        for (int g0 = 0; g0 < k_pairs; g0 += geo_batch) {
            const int gc = min(geo_batch, k_pairs - g0);
            __syncthreads();
            if (g0 > 0 || k_pairs > kGeoPairs) stage_geometry(g0, gc);        // otherwise still valid from pass 1
            for (int q0 = 0; q0 < gc; q0 += P) {
                const int pc = min(P, gc - q0);
                stage_chunk(q0, pc);
                __syncthreads();
                for (int r0 = 0; r0 < pc; r0 += kWarps) {
                    const int nr = min(kWarps, pc - r0);
                    if (wid < nr) {
                        const float* cj = p.c_all + (size_t)geo_j[q0 + r0 + wid] * W;   // every atom is a centre, in order
                        for (int e = lane; e < W; e += 32) {
                            const int r = e / LM;
                            c_copy[r * LMP + (e - r * LM)] = __ldg(cj + e);
                        }
                        __syncwarp();
                        const float4* wSD = sSD4 + (r0 + wid) * LMP;
                        float4* wUV = sUV + wid * NI;
                        if (SN <= 16) {
                            // lane <-> (nu n', half): half 0 accumulates (U, Vx), half 1 (Vy, Vz)
                            const int sn = lane >> 1, half = lane & 1;
                            if (sn < SN) {
                                const float* cp = c_copy + sn * LMP;
                                const float2* hp = reinterpret_cast<const float2*>(wSD) + half;
                                float2* up = reinterpret_cast<float2*>(wUV + sn * L1) + half;
#pragma unroll
                                for (int l = 0; l <= L; ++l) {
                                    float2 acc = make_float2(0.f, 0.f);
#pragma unroll
                                    for (int m = 0; m <= 2 * l; ++m) {
                                        const float cv = cp[l * l + m];
                                        const float2 h = hp[2 * (l * l + m)];
                                        acc.x = fmaf(cv, h.x, acc.x); acc.y = fmaf(cv, h.y, acc.y);
                                    }
                                    const float fl = ((l & 1) ? o_scale : -o_scale) * __ldg(p.kl + l);
                                    up[2 * l] = make_float2(fl * acc.x, fl * acc.y);
                                }
                            }
                        } else {
                            for (int sn = lane; sn < SN; sn += 32) {
                                const float* cp = c_copy + sn * LMP;
#pragma unroll
                                for (int l = 0; l <= L; ++l) {
                                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                                    for (int m = 0; m <= 2 * l; ++m) {
                                        const float cv = cp[l * l + m];
                                        const float4 h = wSD[l * l + m];
                                        acc.x = fmaf(cv, h.x, acc.x); acc.y = fmaf(cv, h.y, acc.y);
                                        acc.z = fmaf(cv, h.z, acc.z); acc.w = fmaf(cv, h.w, acc.w);
                                    }
                                    const float fl = ((l & 1) ? o_scale : -o_scale) * __ldg(p.kl + l);
                                    wUV[sn * L1 + l] = make_float4(fl * acc.x, fl * acc.y, fl * acc.z, fl * acc.w);
                                }
                            }
                        }
                    }
                    __syncthreads();
                    for (int grp = 0; grp < n_groups; ++grp) {
                        if (!in_registers) {
#pragma unroll
                            for (int k = 0; k < kSlots; ++k) {
                                const int x = (grp * kSlots + k) * kThreads + tid;
                                sf[k] = -1;
                                if (x < NZ) {
                                    decode(x, sf[k], sgA[k], suA[k], sgB[k], suB[k]);
                                    ax[k] = row[sf[k]]; ay[k] = row[(size_t)F + sf[k]]; az[k] = row[(size_t)2 * F + sf[k]];
                                }
                            }
                        }
                        for (int w = 0; w < nr; ++w) {
                            const int g = q0 + r0 + w;
                            if (!(geo_i[g].z & 256)) continue;                 // an image of a itself: part of its own row already
                            const float4 d = geo_d[g];
                            const float2* wG = sG2 + (r0 + w) * NCH;
                            const float4* UV = sUV + w * NI;
#pragma unroll
                            for (int k = 0; k < kSlots; ++k) {
                                if (sf[k] < 0) continue;
                                const float2 g1 = wG[sgA[k]];
                                const float4 u1 = UV[suA[k]];
                                float t = g1.y * u1.x;
                                if (sgB[k] >= 0) {
                                    const float2 g2 = wG[sgB[k]];
                                    const float4 u2 = UV[suB[k]];
                                    t = fmaf(g2.y, u2.x, t);
                                    ax[k] = fmaf(g2.x, u2.y, ax[k]); ay[k] = fmaf(g2.x, u2.z, ay[k]); az[k] = fmaf(g2.x, u2.w, az[k]);
                                }
                                ax[k] = fmaf(g1.x, u1.y, fmaf(t, d.x, ax[k]));
                                ay[k] = fmaf(g1.x, u1.z, fmaf(t, d.y, ay[k]));
                                az[k] = fmaf(g1.x, u1.w, fmaf(t, d.z, az[k]));
                            }
                        }
                        if (!in_registers) {
#pragma unroll
                            for (int k = 0; k < kSlots; ++k)
                                if (sf[k] >= 0) { row[sf[k]] = ax[k]; row[(size_t)F + sf[k]] = ay[k]; row[(size_t)2 * F + sf[k]] = az[k]; }
                        }
                    }
                    __syncthreads();
                }
            }
        }
        if (in_registers) {
#pragma unroll
            for (int k = 0; k < kSlots; ++k)
                if (sf[k] >= 0) { row[sf[k]] += ax[k]; row[(size_t)F + sf[k]] += ay[k]; row[(size_t)2 * F + sf[k]] += az[k]; }
        }
        return;
    }
    // fold K_l into c for pass 2
    if (!CC)
        for (int e = tid; e < W; e += kThreads) {
            const int row = e / LM, lm = e - row * LM;
            c_t[row * LMP + lm] *= __ldg(p.kl + __ldg(p.l_of_lm + lm));
        }

    // =========================== pass 2: the Jacobian rows ===========================
    const int NI = S * NCH, SN = S * NMAX;
    // whether the zero blocks of a row can go out as bulk copies: every block boundary, the plane pitch and the
    // row start must sit on 16 bytes
    const bool bulk_ok = !CC && ((((NMAX * (NMAX + 1) / 2) * L1) | (NMAX * NCH) | RW) & 3) == 0 &&
                         (reinterpret_cast<size_t>(p.out_jac) & 15) == 0;
    // coefficient mode: table lm -> l in the (now idle) space of the D tiles; the loop below starts with a barrier
    int* lm_to_l = reinterpret_cast<int*>(smem + lay.wUV);
    if (CC)
        for (int e = tid; e < LM; e += kThreads) lm_to_l[e] = __ldg(p.l_of_lm + e);
    float4* wUV = reinterpret_cast<float4*>(smem + lay.wUV) + wid * NI;       // [nu][n'][l]

    // Product rule of one pair (Eq. 5).  Lanes take consecutive features of the row in sweeps that
    // are aligned to the row's start, so every warp store covers whole 32-byte sectors of each of the
    // three direction planes (sectors written in two pieces halve the achievable write bandwidth).
    // Feature (mu, nu, n1, n2, l) of a neighbour of species Z:
    //   mu == Z:  G_{n1 l} V^nu_{n2 l} + Ghat_{n1 l} U^nu_{n2 l} d      (grad c^mu_{n1 l}) c^nu_{n2 l}
    //   nu == Z:  G_{n2 l} V^mu_{n1 l} + Ghat_{n2 l} U^mu_{n1 l} d      c^mu_{n1 l} (grad c^nu_{n2 l})
    // (both when mu == nu == Z, zero when neither).  Stores the row, or adds to it when another
    // image of the same atom already wrote it.
    auto product_rule = [&](auto acc_tag, int Z, float4 d, const float2* wG, float* out) {
        constexpr bool ACC = decltype(acc_tag)::value;
        const int PS = RW, PS2 = 2 * RW;                      // stride between the three direction planes
        // position of the row start inside a 128-byte line, in floats: sweeps start on line boundaries
        // where the row allows it (a warp store that straddles two lines costs two L1 wavefronts)
        const int a_line = (int)((reinterpret_cast<size_t>(out) >> 2) & 31);
        auto put = [&](int f, float vx, float vy, float vz) {
            if (ACC) { out[f] += vx; out[PS + f] += vy; out[PS2 + f] += vz; }
            else { out[f] = vx; out[PS + f] = vy; out[PS2 + f] = vz; }
        };
        int lo = 0;
        for (int mu = 0; mu < S; ++mu) {
            for (int nu = mu; nu < (o_cross ? S : mu + 1); ++nu) {
                const int hi = lo + ((mu == nu) ? (NMAX * (NMAX + 1) / 2) * L1 : NMAX * NCH);
                const int first = ((lo + a_line) & ~31) - a_line;
                if (mu != Z && nu != Z) {
                    if (o_compact) continue;                  // compact rows hold only the blocks that involve Z
                    if (!ACC) {
                        if (bulk_ok) {
                            // structural zeros: the lanes hand the plane segments (pieces of at most kZeroWords) to the copy engine
                            const int parts = (hi - lo + kZeroWords - 1) / kZeroWords;
                            for (int idx = lane; idx < 3 * parts; idx += 32) {
                                const int k = idx / parts, f = lo + (idx - k * parts) * kZeroWords;
                                bulk_store(out + k * PS + f, zero_buf, 4u * (unsigned)min(kZeroWords, hi - f));
                            }
                        } else {
                            for (int f = first + lane; f < hi; f += 32)
                                if (f >= lo) put(f, 0.f, 0.f, 0.f);
                        }
                    }
                } else if (mu == nu && NMAX_T != 0 && NMAX_T <= 4) {
                    // small n_max: lanes on the columns (n2, l) with their own operand in registers, rows n1 <= n2
                    // in turn: fewer instructions than the table-driven sweeps below, stores contiguous but not
                    // sector-aligned (3 to 6 % faster up to n_max = 4, slower from 5 on)
                    const float4* UVz = wUV + Z * NCH;
                    for (int j0 = 0; j0 < NCH; j0 += 32) {
                        const int j = j0 + lane;
                        if (j >= NCH) break;
                        const int n2 = j / L1, l = j - n2 * L1;
                        const float2 gj = wG[j];
                        const float4 uj = UVz[j];
                        float* o = out + lo + j;
#pragma unroll
                        for (int n1 = 0; n1 < NMAX_BOUND; ++n1) {
                            if (n1 >= NMAX || n1 * L1 > min(j0 + 31, NCH - 1)) break;           // no lane of this round has n2 >= n1
                            const int rel = (n1 * NMAX - n1 * (n1 - 1) / 2) * L1 - n1 * L1;     // row start minus n1 L1
                            if (n1 <= n2) {
                                const float2 gi = wG[n1 * L1 + l];
                                const float4 ui = UVz[n1 * L1 + l];
                                const float t = fmaf(gi.y, uj.x, gj.y * ui.x);
                                const float vx = fmaf(gi.x, uj.y, fmaf(gj.x, ui.y, t * d.x));
                                const float vy = fmaf(gi.x, uj.z, fmaf(gj.x, ui.z, t * d.y));
                                const float vz = fmaf(gi.x, uj.w, fmaf(gj.x, ui.w, t * d.z));
                                if (ACC) { o[rel] += vx; o[PS + rel] += vy; o[PS2 + rel] += vz; }
                                else { o[rel] = vx; o[PS + rel] = vy; o[PS2 + rel] = vz; }
                            }
                        }
                    }
                } else if (mu == nu && NMAX_T != 0) {
                    // compile-time n_max: the sweeps are unrolled in full, so that the table index and the three store
                    // addresses of a sweep are constants off pointers formed once per block
                    const float4* UVz = wUV + Z * NCH;
                    constexpr int TRI_T = (NMAX_BOUND * (NMAX_BOUND + 1) / 2) * L1;
                    constexpr int SWEEPS = (TRI_T + 62) / 32;                   // the block and up to 31 floats in front of it
                    const int e0 = first - lo + lane;                           // -31 .. 31: place of this lane's first feature in the block
                    const unsigned short* dp = tri_dec + e0;
                    float* const o0 = out + (first + lane);
                    float* const o1 = o0 + PS;
                    float* const o2 = o0 + PS2;
#pragma unroll
                    for (int k = 0; k < SWEEPS; ++k) {
                        const int e = e0 + 32 * k;
                        if ((k > 0 || e >= 0) && (32 * k + 31 < TRI_T || e < TRI_T)) {
                            const unsigned dec = dp[32 * k];                    // (n1 L1 + l) | (n2 L1 + l) << 8
                            const int iA = dec & 255, iB = dec >> 8;
                            const float2 g1 = wG[iA], g2 = wG[iB];
                            const float4 u1 = UVz[iA], u2 = UVz[iB];
                            const float t = fmaf(g1.y, u2.x, g2.y * u1.x);      // Ghat_n1 U_n2 + Ghat_n2 U_n1
                            const float vx = fmaf(g1.x, u2.y, fmaf(g2.x, u1.y, t * d.x)), vy = fmaf(g1.x, u2.z, fmaf(g2.x, u1.z, t * d.y)),
                                        vz = fmaf(g1.x, u2.w, fmaf(g2.x, u1.w, t * d.z));
                            if (ACC) { o0[32 * k] += vx; o1[32 * k] += vy; o2[32 * k] += vz; }
                            else { o0[32 * k] = vx; o1[32 * k] = vy; o2[32 * k] = vz; }
                        }
                    }
                } else if (mu == nu) {
                    const float4* UVz = wUV + Z * NCH;
#pragma unroll kTriUnroll
                    for (int f = first + lane; f < hi; f += 32) {
                        if (f < lo) continue;
                        const unsigned dec = tri_dec[f - lo];                 // (n1 L1 + l) | (n2 L1 + l) << 8
                        const int iA = dec & 255, iB = dec >> 8;
                        const float2 g1 = wG[iA], g2 = wG[iB];
                        const float4 u1 = UVz[iA], u2 = UVz[iB];
                        const float t = fmaf(g1.y, u2.x, g2.y * u1.x);      // Ghat_n1 U_n2 + Ghat_n2 U_n1
                        put(f, fmaf(g1.x, u2.y, fmaf(g2.x, u1.y, t * d.x)), fmaf(g1.x, u2.z, fmaf(g2.x, u1.z, t * d.y)),
                            fmaf(g1.x, u2.w, fmaf(g2.x, u1.w, t * d.z)));
                    }
                } else if (kCrossTable) {
                    // rows that do not all start on a sector boundary: sweeps aligned to the row start of the Jacobian
                    // row, as in the same-species block, with the two operand indices of a feature from a table
                    const bool first_term = (mu == Z);                        // which factor belongs to the moved atom
                    const float4* UVo = wUV + (first_term ? nu : mu) * NCH;
                    constexpr int SQ_T = NMAX_BOUND * NMAX_BOUND * L1, SWEEPS = (SQ_T + 62) / 32, kUnroll = 8;
                    const int e0 = first - lo + lane;                           // -31 .. 31
                    for (int k0 = 0; k0 < SWEEPS; k0 += kUnroll) {
                        const unsigned short* dp = x_dec + e0 + 32 * k0;
                        float* const o0 = out + (first + lane + 32 * k0);
                        float* const o1 = o0 + PS;
                        float* const o2 = o0 + PS2;
#pragma unroll
                        for (int kk = 0; kk < kUnroll; ++kk) {
                            const int e = e0 + 32 * (k0 + kk);
                            if (k0 + kk < SWEEPS && e >= 0 && e < SQ_T) {
                                const unsigned dec = dp[32 * kk];
                                const int i1 = dec & 255, j = dec >> 8;
                                const float2 g = wG[first_term ? i1 : j];
                                const float4 u = UVo[first_term ? j : i1];
                                const float t = g.y * u.x;
                                const float vx = fmaf(g.x, u.y, t * d.x), vy = fmaf(g.x, u.z, t * d.y), vz = fmaf(g.x, u.w, t * d.z);
                                if (ACC) { o0[32 * kk] += vx; o1[32 * kk] += vy; o2[32 * kk] += vz; }
                                else { o0[32 * kk] = vx; o1[32 * kk] = vy; o2[32 * kk] = vz; }
                            }
                        }
                    }
                } else if ((NCH & 7) == 0 || (NMAX_T > 8 && (NCH & 3) == 0) || (NMAX_T != 0 && NMAX_T <= 8)) {
                    // Cross-species block: rows n1 of n_ch floats follow each other.  A lane keeps one position i of
                    // a window of about n_ch floats, so its (n2, l) is fixed and the operand that depends on (n2, l)
                    // stays in registers over the unrolled n1 loop.
                    //  * n_ch a multiple of 8: every row starts at the same offset inside a 32-byte sector; the
                    //    windows start `shift` floats before the row starts, on sector boundaries, and the lanes in
                    //    front of a row start (i < shift) serve the tail of the previous row.
                    //  * n_ch a multiple of 4 only: the offset alternates between two values, so even and odd rows
                    //    are done in two passes, each with its own shift and window length (taken from n_max = 9
                    //    on, where it gains 7 to 8 %; with few rows per pass the set-up costs more than it saves,
                    //    and a window must not be shorter than its shift).
                    //  * otherwise (taken up to n_max = 8): no shift, lanes sit on the columns themselves; the warp
                    //    stores are contiguous but not sector-aligned, which still beats decoding every feature by 2 to
                    //    14 %; from n_max = 10 on it loses (up to 24 %), so those keep the aligned sweeps below.
                    const bool first_term = (mu == Z);
                    const float4* UVo = wUV + (first_term ? nu : mu) * NCH;
                    const int T = (NCH & 7) == 0 ? 1 : ((NMAX_T > 8 && (NCH & 3) == 0) ? 2 : ((NMAX_T > 8 && (NCH & 3) == 0) ? 4 : 0));
                    const int TT = T ? T : 1;
#pragma unroll
                    for (int pp = 0; pp < 4; ++pp) {
                        if (pp >= TT) break;
                        const int shift = T ? ((a_line + lo + pp * NCH) & 7) : 0;
                        const int wlen = NCH + shift - (T ? ((a_line + lo + (pp + 1) * NCH) & 7) : 0);
                        for (int i0 = 0; i0 < wlen; i0 += 32) {
                            const int i = i0 + lane;
                            if (i >= wlen) break;
                            const bool prev = i < shift;                          // belongs to row n1 - 1
                            const int j = prev ? i - shift + NCH : i - shift;      // n2 L1 + l
                            const int l = j % L1;
                            float* o = out + (lo - shift + i);
                            if (first_term) {
                                const float4 u = UVo[j];
                                const float xx = u.x * d.x, xy = u.x * d.y, xz = u.x * d.z;
                                const float2* gp = wG + l - (prev ? L1 : 0);
#pragma unroll
                                for (int k = 0; k <= NMAX_BOUND; ++k) {
                                    const int n1 = pp + k * TT;
                                    if (n1 > NMAX) break;
                                    if (prev ? (n1 >= 1) : (n1 < NMAX)) {
                                        const float2 g = gp[n1 * L1];
                                        const float vx = fmaf(g.x, u.y, g.y * xx), vy = fmaf(g.x, u.z, g.y * xy), vz = fmaf(g.x, u.w, g.y * xz);
                                        if (ACC) { o[n1 * NCH] += vx; o[PS + n1 * NCH] += vy; o[PS2 + n1 * NCH] += vz; }
                                        else { o[n1 * NCH] = vx; o[PS + n1 * NCH] = vy; o[PS2 + n1 * NCH] = vz; }
                                    }
                                }
                            } else {
                                const float2 g = wG[j];
                                const float gx = g.y * d.x, gy = g.y * d.y, gz = g.y * d.z;
                                const float4* up = UVo + l - (prev ? L1 : 0);
#pragma unroll
                                for (int k = 0; k <= NMAX_BOUND; ++k) {
                                    const int n1 = pp + k * TT;
                                    if (n1 > NMAX) break;
                                    if (prev ? (n1 >= 1) : (n1 < NMAX)) {
                                        const float4 u = up[n1 * L1];
                                        const float vx = fmaf(g.x, u.y, gx * u.x), vy = fmaf(g.x, u.z, gy * u.x), vz = fmaf(g.x, u.w, gz * u.x);
                                        if (ACC) { o[n1 * NCH] += vx; o[PS + n1 * NCH] += vy; o[PS2 + n1 * NCH] += vz; }
                                        else { o[n1 * NCH] = vx; o[PS + n1 * NCH] = vy; o[PS2 + n1 * NCH] = vz; }
                                    }
                                }
                            }
                        }
                    }
                } else {
                    // block index e = n1 NCH + n2 L1 + l; the radial factor belongs to the neighbour's
                    // species, U/V to the other one
                    const bool first_term = (mu == Z);
                    const float4* UVo = wUV + (first_term ? nu : mu) * NCH;
#pragma unroll 2
                    for (int f = first + lane; f < hi; f += 32) {
                        if (f < lo) continue;
                        const int e = f - lo;
                        const int n1 = (int)__umulhi((unsigned)e, p.nch_magic);
                        const int j = e - n1 * NCH;                           // n2 L1 + l
                        const int i1 = n1 * L1 + (j % L1);                    // n1 L1 + l
                        const float2 g = wG[first_term ? i1 : j];
                        const float4 u = UVo[first_term ? j : i1];
                        const float t = g.y * u.x;
                        put(f, fmaf(g.x, u.y, t * d.x), fmaf(g.x, u.z, t * d.y), fmaf(g.x, u.w, t * d.z));
                    }
                }
                lo = hi;
            }
        }
        // compact rows are padded to a multiple of eight floats: the padding is written as zeros
        if (o_compact && !ACC)
            for (int f = lo + lane; f < RW; f += 32) put(f, 0.f, 0.f, 0.f);
    };

    // Coefficient mode: the row of a neighbour of species Z is grad c^Z_nlm = G_nl grad S_lm + Ghat_nl d S_lm
    // (Eq. 14 / Eq. 23) in the block of Z and zero in the other blocks, written in aligned sweeps as above.
    auto coeff_rule = [&](auto acc_tag, int Z, float4 d, const float2* wG, const float4* wSD, float* out) {
        constexpr bool ACC = decltype(acc_tag)::value;
        const int a_line = (int)((reinterpret_cast<size_t>(out) >> 2) & 31);
        for (int s = 0; s < S; ++s) {
            if (ACC && s != Z) continue;
            const int lo = s * NE, hi = lo + NE;
            const int first = ((lo + a_line) & ~31) - a_line;
            for (int f = first + lane; f < hi; f += 32) {
                if (f < lo) continue;
                float vx = 0.f, vy = 0.f, vz = 0.f;
                if (s == Z) {
                    const int e = f - lo, n = e / LM, lm = e - n * LM;
                    const int l = lm_to_l[lm];                            // lm = l^2 + l + m
                    const float2 g = wG[n * L1 + l];
                    const float4 h = wSD[lm];
                    const float t = g.y * h.x;
                    vx = fmaf(g.x, h.y, t * d.x); vy = fmaf(g.x, h.z, t * d.y); vz = fmaf(g.x, h.w, t * d.z);
                }
                if (ACC) { out[f] += vx; out[W + f] += vy; out[2 * W + f] += vz; }
                else { out[f] = vx; out[W + f] = vy; out[2 * W + f] = vz; }
            }
        }
    };

    // everything one warp does for one pair of the staged chunk
    auto do_pair = [&](int g, int pr) {
        const int4 gi = geo_i[g];
        const int rw = gi.w;
        const int row = rw & kRowMask;
        const int Z = gi.z & 255;
        const float4 d = geo_d[g];
        const float2* wG = sG2 + pr * NCH;
        const float4* wSD = sSD4 + pr * LMP;
        __syncwarp();
        // ---- U, V for every (nu, n', l) ----
        if (CC) {
        } else if (SN <= 16) {
            // lane <-> (nu n', half): half 0 accumulates (U, Vx), half 1 (Vy, Vz)
            const int sn = lane >> 1, half = lane & 1;
            if (sn < SN) {
                const float* cp = c_t + sn * LMP;
                const float2* hp = reinterpret_cast<const float2*>(wSD) + half;
                float2* up = reinterpret_cast<float2*>(wUV + sn * L1) + half;
#pragma unroll
                for (int l = 0; l <= L; ++l) {
                    float2 acc = make_float2(0.f, 0.f);
#pragma unroll
                    for (int m = 0; m <= 2 * l; ++m) {
                        const float cv = cp[l * l + m];
                        const float2 h = hp[2 * (l * l + m)];
                        acc.x = fmaf(cv, h.x, acc.x); acc.y = fmaf(cv, h.y, acc.y);
                    }
                    up[2 * l] = acc;
                }
            }
        } else {
            for (int sn = lane; sn < SN; sn += 32) {
                const float* cp = c_t + sn * LMP;
#pragma unroll
                for (int l = 0; l <= L; ++l) {
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int m = 0; m <= 2 * l; ++m) {
                        const float cv = cp[l * l + m];
                        const float4 h = wSD[l * l + m];
                        acc.x = fmaf(cv, h.x, acc.x); acc.y = fmaf(cv, h.y, acc.y);
                        acc.z = fmaf(cv, h.z, acc.z); acc.w = fmaf(cv, h.w, acc.w);
                    }
                    wUV[sn * L1 + l] = acc;
                }
            }
        }
        __syncwarp();
        float* out = p.out_jac + (size_t)(row_base + row) * 3 * RW;
        if (rw & kRowContinuation) {
            if (CC) coeff_rule(std::true_type{}, Z, d, wG, wSD, out);
            else product_rule(std::true_type{}, Z, d, wG, out);
        } else {
            if (lane == 0) p.row_atom[row_base + row] = geo_j[g];
            if (CC) coeff_rule(std::false_type{}, Z, d, wG, wSD, out);
            else product_rule(std::false_type{}, Z, d, wG, out);
            if (bulk_ok) bulk_commit();
        }
    };

    const int PW = P / kWarps;             // pairs a warp stages for itself (the staging area holds P)
    for (int g0 = 0; g0 < k_pairs; g0 += geo_batch) {
        const int gc = min(geo_batch, k_pairs - g0);
        __syncthreads();
        if (g0 > 0 || k_pairs > kGeoPairs) special = stage_geometry(g0, gc);     // otherwise still valid from pass 1
        // (measured on the 1000-molecule cluster: 1 to 4 % faster from n_max = 8 on up to l_max = 8; with fewer
        // channels than lanes, or more columns m than the eight lanes of a pair, the staging by the whole CTA wins)
        constexpr bool kPrivate = !CC && NMAX_T >= 8 && L <= 8;      // (the coefficient rows are cheap per pair: staging by the CTA wins there)
        if (kPrivate && !special && PW >= 1) {
            // Every pair has a row of its own: the warps work without one another.  Warp w takes the pairs w, w + 8,
            // ... of the batch, PW at a time: it stages their radial factors (lanes on channels) and harmonics (eight
            // lanes per pair, on the columns m of the recursion) in its own part of the staging area, then writes
            // their rows.  No CTA barrier until the next batch of geometry.
            const int slot0 = wid * PW;
            for (int gw = wid; gw < gc; gw += PW * kWarps) {
                const int nb = min(PW, (gc - gw + kWarps - 1) / kWarps);
                __syncwarp();
                for (int pr = 0; pr < nb; ++pr) {
                    const int g = gw + pr * kWarps;
                    const int4 gi = geo_i[g];
                    const float t = __int_as_float(gi.y);
                    const float rinv_h = (float)p.inv_h / geo_d[g].w;
                    float2* mG = sG2 + (slot0 + pr) * NCH;
                    if (o_pw) {
                        const float2 w = geo_w[g];
                        for (int ch = lane; ch < NCH; ch += 32) {
                            float v, dv;
                            radial_lookup(p.table, gi.x, NCH, ch, t, v, dv);
                            mG[ch] = make_float2(v * w.x, fmaf(dv * rinv_h, w.x, v * w.y));
                        }
                    } else {
                        for (int ch = lane; ch < NCH; ch += 32) {
                            float v, dv;
                            radial_lookup(p.table, gi.x, NCH, ch, t, v, dv);
                            mG[ch] = make_float2(v, dv * rinv_h);
                        }
                    }
                }
                {
                    const int pr = lane >> 3;
                    if (pr < nb) {
                        const float4 d = geo_d[gw + pr * kWarps];
                        for (int m = lane & 7; m <= L; m += 8)
                            harmonics_column(L, m, d.x, d.y, d.z, d.w * d.w, sSD4 + (slot0 + pr) * LMP);
                    }
                }
                __syncwarp();
                for (int pr = 0; pr < nb; ++pr) do_pair(gw + pr * kWarps, slot0 + pr);
            }
            continue;
        }
        // Images of one atom share a row (or the staging area holds fewer pairs than there are warps): staged by the
        // whole CTA in chunks of equal size, a multiple of the warp count.
        const int n_chunks = (gc + P - 1) / P;
        const int PB = min(P, (((gc + n_chunks - 1) / n_chunks) + kWarps - 1) & ~(kWarps - 1));
        for (int q0 = 0; q0 < gc; q0 += PB) {
            const int pc = min(PB, gc - q0);
            stage_chunk(q0, pc);
            __syncthreads();
            if (!special) {
                for (int pr = wid; pr < pc; pr += kWarps) do_pair(q0 + pr, pr);
            } else {
                // images of one atom must stay with one warp, in order;
                // images of the centre itself do not move relative to it and are skipped
                for (int pr = 0; pr < pc; ++pr) {
                    const int rw = geo_i[q0 + pr].w;
                    if ((rw & kRowSelfImage) || ((rw & kRowMask) & (kWarps - 1)) != wid) continue;
                    do_pair(q0 + pr, pr);
                }
            }
            __syncthreads();
        }
    }
    // the zeros in shared memory must outlive the copies that read them
    if (bulk_ok) bulk_wait_read();
}

}  // namespace soap
