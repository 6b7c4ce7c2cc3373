// The fused per-centre kernel: one CTA owns one centre atom and produces its
// descriptor row (Eq. 4) and, in the derivative build, all of its Jacobian
// rows (Eq. 5).  Nothing per pair ever goes to HBM: radial factors, solid
// harmonics and the precontracted U/V live in shared memory; the expansion
// coefficients c^mu_nlm of the centre stay in shared memory for the CTA's life.
//
// Per pair (displacement d = r_j + T - r_i, species Z of j):
//   c^Z_nlm        += G_nl(|d|) S_lm(d)                               (Eq. 13 / 18)
//   grad_j c^Z_nlm  = G_nl grad S_lm + Ghat_nl d S_lm,  Ghat = G'/|d|  (Eq. 14 / 23)
// with S_lm = r^l Y_lm the real solid harmonic and G_nl, G'_nl read from the
// degree-5 tables.
//   Pass 1 (whole CTA per chunk of pairs) accumulates c and D = sum_j grad_j c;
//   the centre's own Jacobian row is minus the sum over its neighbours, which is
//   a contraction of D with c.
//   Pass 2 (one warp per pair, no block barriers) forms U^nu_{n'l} = K_l sum_m
//   S_lm c^nu_{n'lm} and V likewise with grad S, after which every output
//   element of Eq. 5 is two fused multiply-adds per term, and streams the row
//   out with lanes on consecutive features.
// l_max is a template parameter so that the harmonic recursions unroll and the
// index arithmetic folds; n_max and the species count stay run-time values.
#pragma once
#include "soap_device.cuh"

namespace soap {

// Real solid harmonics S_{l,+m}, S_{l,-m} (and gradients) for one (l, m >= 0):
//   S_{l,+m} = a_lm Q_l^m Re (x+iy)^m,   S_{l,-m} = a_lm Q_l^m Im (x+iy)^m,
//   Q_l^m = r^(l-m) d^m P_l(t)/dt^m at t = z/r, by the recurrence
//   (l-m) Q_l^m = (2l-1) z Q_{l-1}^m - (l+m-1) r^2 Q_{l-2}^m,  Q_m^m = (2m-1)!!,
//   dQ_l^m/dx = -x Q_{l-1}^{m+1},  dQ_l^m/dy = -y Q_{l-1}^{m+1},  dQ_l^m/dz = (l+m) Q_{l-1}^m.
// Every lane runs the same unrolled, predicated recurrences for its own (l, m).
template <int L, bool GRAD>
__device__ __forceinline__ void solid_harmonic_item(float x, float y, float z, float r2, int l, int m,
                                                    const float* __restrict__ anorm, const float* __restrict__ dfact,
                                                    const float* __restrict__ inv_int,
                                                    float4& plus, float4& minus) {
    float cm = 1.f, sm = 0.f, cp = 0.f, sp = 0.f;          // (x+iy)^m and (x+iy)^(m-1)
#pragma unroll
    for (int t = 0; t < L; ++t)
        if (t < m) {
            cp = cm; sp = sm;
            const float cn = x * cm - y * sm;
            sm = x * sm + y * cm;
            cm = cn;
        }
    float qa = __ldg(dfact + m), qb = 0.f;                  // Q_ll^m, Q_{ll-1}^m
    float qc = 0.f, qd = 0.f;                               // Q_ll^{m+1}, Q_{ll-1}^{m+1} (up to ll = l-1)
    if (GRAD && m + 1 <= l - 1) qc = __ldg(dfact + m + 1);
#pragma unroll
    for (int ll = 1; ll <= L; ++ll) {
        if (ll > m && ll <= l) {
            const float qn = ((2 * ll - 1) * z * qa - (ll + m - 1) * r2 * qb) * __ldg(inv_int + ll - m);
            qb = qa; qa = qn;
        }
        if (GRAD && ll > m + 1 && ll <= l - 1) {
            const float qn = ((2 * ll - 1) * z * qc - (ll + m) * r2 * qd) * __ldg(inv_int + ll - m - 1);
            qd = qc; qc = qn;
        }
    }
    const float a = __ldg(anorm + l * (l + 1) / 2 + m);
    const float aq = a * qa;
    if (!GRAD) {
        plus.x = aq * cm;
        minus.x = aq * sm;
        return;
    }
    const float qz = (l > m) ? a * (l + m) * qb : 0.f;      // a dQ/dz
    const float qx = a * qc;                                // a Q_{l-1}^{m+1} (0 when it does not exist)
    const float mq = m * aq;
    plus = make_float4(aq * cm, -x * qx * cm + mq * cp, -y * qx * cm - mq * sp, qz * cm);
    minus = make_float4(aq * sm, -x * qx * sm + mq * sp, -y * qx * sm + mq * cp, qz * sm);
}

// Degree-5 table lookup: value and derivative with respect to the interval coordinate t.
__device__ __forceinline__ void radial_lookup(const float* __restrict__ table, int qi, int n_ch, int ch, float t,
                                              float& v, float& dv) {
    const float2* cf = reinterpret_cast<const float2*>(table + ((size_t)qi * n_ch + ch) * 6);
    const float2 a = __ldg(cf), b = __ldg(cf + 1), c = __ldg(cf + 2);
    v = c.y; dv = 0.f;
    dv = fmaf(dv, t, v); v = fmaf(v, t, c.x);
    dv = fmaf(dv, t, v); v = fmaf(v, t, b.y);
    dv = fmaf(dv, t, v); v = fmaf(v, t, b.x);
    dv = fmaf(dv, t, v); v = fmaf(v, t, a.y);
    dv = fmaf(dv, t, v); v = fmaf(v, t, a.x);
}

template <bool DERIV, int L>
__global__ void __launch_bounds__(kThreads, DERIV ? 3 : 4)
center_kernel(const CenterParams p) {
    constexpr int L1 = L + 1, LM = L1 * L1, NQ = L1 * (L1 + 1) / 2;
    constexpr int KE = (16 * LM + kThreads - 1) / kThreads < kMaxElemPerThread ? (16 * LM + kThreads - 1) / kThreads
                                                                                : kMaxElemPerThread;
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const long long c_idx = blockIdx.x;
    // a failed neighbour build or an undersized output: write nothing
    if (p.pair_ptr[p.n_centers] > p.pair_capacity) return;
    if (DERIV && p.row_ptr[p.n_centers] > p.row_capacity) {
        if (c_idx == 0 && tid == 0) atomicOr(&p.counters->status, kStatusRowCapacity);
        return;
    }
    const int S = p.S, NMAX = p.n_max, NCH = NMAX * L1, NE = NMAX * LM, CT = S * NE, P = p.P, F = p.F;
    const SmemLayout lay = make_layout(S, NMAX, L, P, DERIV);
    float* c_t = smem + lay.c;
    float4* geo_d = reinterpret_cast<float4*>(smem + lay.geo);             // [GP] dx, dy, dz, r
    int4* geo_i = reinterpret_cast<int4*>(smem + lay.geo + 4 * kGeoPairs);   // [GP] interval, t bits, species|moving<<8, row word
    float* D_t = smem + lay.D;                                             // [3][CT]           (pass 1)
    float* sS = smem + lay.sSD;                                            // [P][LM]           (pass 1, descriptor build)
    float4* sSD4 = reinterpret_cast<float4*>(smem + lay.sSD);              // [P][LM]           (pass 1, derivative build)
    float* sG1 = smem + lay.sG;
    float2* sG2 = reinterpret_cast<float2*>(smem + lay.sG);                // [P][NCH]

    const int ci = p.centers ? p.centers[c_idx] : (int)c_idx;
    const float xi = p.pos[3 * (long long)ci], yi = p.pos[3 * (long long)ci + 1], zi = p.pos[3 * (long long)ci + 2];
    const int zi_species = p.species_idx[ci];
    const long long pair_base = p.pair_ptr[c_idx];
    const int k_pairs = (int)(p.pair_ptr[c_idx + 1] - pair_base);
    const bool periodic = p.geom.pbc[0] | p.geom.pbc[1] | p.geom.pbc[2];

    for (int e = tid; e < CT * (DERIV ? 4 : 1); e += kThreads) {
        if (e < CT) c_t[e] = 0.f; else D_t[e - CT] = 0.f;
    }

    // elements (n, lm) this thread accumulates in pass 1
    int el_lm[KE], el_ch[KE];
#pragma unroll
    for (int k = 0; k < KE; ++k) {
        const int e = tid + k * kThreads;
        const int n = e / LM, lm = e - n * LM;
        el_lm[k] = e < NE ? lm : -1;
        el_ch[k] = n * L1 + __ldg(p.l_of_lm + lm);
    }

    // ---- geometry of up to kGeoPairs pairs, one thread each ----
    auto stage_geometry = [&](int g0, int gc) {
        if (tid < gc) {
            const unsigned long long key = p.pair_key[pair_base + g0 + tid];
            const int j = key_atom(key);
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
            geo_d[tid] = make_float4((float)dx, (float)dy, (float)dz, (float)r);
            const int rw = p.pair_row[pair_base + g0 + tid];
            // interval and offset in the radial table, in fp64 so that the offset keeps its digits
            const double u = r * (double)p.inv_h;
            const int qi = min((int)u, p.n_intervals - 1);
            geo_i[tid] = make_int4(qi, __float_as_int((float)(u - qi)),
                                   p.species_idx[j] | ((rw & kRowSelfImage) ? 0 : 256), rw);
        }
    };

    // =========================== pass 1: c (and D) ===========================
    for (int g0 = 0; g0 < k_pairs; g0 += kGeoPairs) {
        const int gc = min(kGeoPairs, k_pairs - g0);
        __syncthreads();
        stage_geometry(g0, gc);
        __syncthreads();
        for (int q0 = 0; q0 < gc; q0 += P) {
            const int pc = min(P, gc - q0);
            // radial factors: warp <-> pair, lane <-> channel
            for (int pr = wid; pr < pc; pr += kWarps) {
                const int4 gi = geo_i[q0 + pr];
                const float t = __int_as_float(gi.y);
                const float rinv_h = p.inv_h / geo_d[q0 + pr].w;
                for (int ch = lane; ch < NCH; ch += 32) {
                    float v, dv;
                    radial_lookup(p.table, gi.x, NCH, ch, t, v, dv);
                    if (DERIV) sG2[pr * NCH + ch] = make_float2(v, dv * rinv_h);
                    else sG1[pr * NCH + ch] = v;
                }
            }
            // solid harmonics: thread <-> (pair, (l, m >= 0))
            for (int idx = tid; idx < pc * NQ; idx += kThreads) {
                const int pr = idx / NQ, t = idx - pr * NQ;
                const int lmp = __ldg(p.lm_of_t + t);
                const int l = lmp >> 4, m = lmp & 15;
                const float4 d = geo_d[q0 + pr];
                float4 plus, minus;
                solid_harmonic_item<L, DERIV>(d.x, d.y, d.z, d.w * d.w, l, m, p.anorm, p.dfact, p.inv_int, plus, minus);
                const int lm0 = l * l + l;
                if (DERIV) {
                    sSD4[pr * LM + lm0 + m] = plus;
                    if (m) sSD4[pr * LM + lm0 - m] = minus;
                } else {
                    sS[pr * LM + lm0 + m] = plus.x;
                    if (m) sS[pr * LM + lm0 - m] = minus.x;
                }
            }
            __syncthreads();
            for (int s = 0; s < S; ++s) {
                float ac[KE], ax[KE], ay[KE], az[KE];
#pragma unroll
                for (int k = 0; k < KE; ++k) ac[k] = ax[k] = ay[k] = az[k] = 0.f;
                bool any = false;
                for (int pr = 0; pr < pc; ++pr) {
                    const int info = geo_i[q0 + pr].z;
                    if ((info & 255) != s) continue;
                    any = true;
                    if (!DERIV) {
#pragma unroll
                        for (int k = 0; k < KE; ++k)
                            if (el_lm[k] >= 0) ac[k] = fmaf(sG1[pr * NCH + el_ch[k]], sS[pr * LM + el_lm[k]], ac[k]);
                    } else {
                        const float4 d = geo_d[q0 + pr];
                        const float mv = (info & 256) ? 1.f : 0.f;   // an image of the centre does not move relative to it
#pragma unroll
                        for (int k = 0; k < KE; ++k)
                            if (el_lm[k] >= 0) {
                                const float2 g = sG2[pr * NCH + el_ch[k]];
                                const float4 h = sSD4[pr * LM + el_lm[k]];
                                ac[k] = fmaf(g.x, h.x, ac[k]);
                                const float gm = g.x * mv, t = g.y * h.x * mv;
                                ax[k] = fmaf(gm, h.y, fmaf(t, d.x, ax[k]));
                                ay[k] = fmaf(gm, h.z, fmaf(t, d.y, ay[k]));
                                az[k] = fmaf(gm, h.w, fmaf(t, d.z, az[k]));
                            }
                    }
                }
                if (any) {
#pragma unroll
                    for (int k = 0; k < KE; ++k)
                        if (el_lm[k] >= 0) {
                            const int e = s * NE + tid + k * kThreads;
                            c_t[e] += ac[k];
                            if (DERIV) { D_t[e] += ax[k]; D_t[CT + e] += ay[k]; D_t[2 * CT + e] += az[k]; }
                        }
                }
            }
            __syncthreads();
        }
    }
    __syncthreads();
    // on-site term: the centre's own Gaussian, l = 0 only (second term of Eq. 13)
    if (tid < NMAX) c_t[(zi_species * NMAX + tid) * LM] += __ldg(p.self_term + tid);
    __syncthreads();

    // ====================== power spectrum, Eq. 4 ======================
    float* desc_row = p.out_desc + (size_t)c_idx * F;
    for (int f = tid; f < F; f += kThreads) {
        const int pk = __ldg(p.feat_pack + f);
        const int n1 = pk & 31, n2 = (pk >> 5) & 31, mu = (pk >> 10) & 15, nu = (pk >> 14) & 15, l = (pk >> 18) & 15;
        const float* a = c_t + (mu * NMAX + n1) * LM + l * l;
        const float* b = c_t + (nu * NMAX + n2) * LM + l * l;
        float acc = 0.f;
        for (int m = 0; m <= 2 * l; ++m) acc = fmaf(a[m], b[m], acc);
        desc_row[f] = __ldg(p.kl + l) * acc;
    }
    if (!DERIV) return;

    // ============ the centre's own row: minus the sum over its neighbours ============
    const long long row_base = p.row_ptr[c_idx];
    const int my_row = p.self_row[c_idx];
    {
        float* out = p.out_jac + (size_t)(row_base + my_row) * 3 * F;
        for (int f = tid; f < F; f += kThreads) {
            const int pk = __ldg(p.feat_pack + f);
            const int n1 = pk & 31, n2 = (pk >> 5) & 31, mu = (pk >> 10) & 15, nu = (pk >> 14) & 15, l = (pk >> 18) & 15;
            const int ia = (mu * NMAX + n1) * LM + l * l, ib = (nu * NMAX + n2) * LM + l * l;
            const float kl = -__ldg(p.kl + l);
            float ax = 0.f, ay = 0.f, az = 0.f;
            for (int m = 0; m <= 2 * l; ++m) {
                const float ca = c_t[ia + m], cb = c_t[ib + m];
                ax = fmaf(D_t[ia + m], cb, fmaf(ca, D_t[ib + m], ax));
                ay = fmaf(D_t[CT + ia + m], cb, fmaf(ca, D_t[CT + ib + m], ay));
                az = fmaf(D_t[2 * CT + ia + m], cb, fmaf(ca, D_t[2 * CT + ib + m], az));
            }
            out[f] = kl * ax; out[(size_t)F + f] = kl * ay; out[(size_t)2 * F + f] = kl * az;
        }
        if (tid == 0) p.row_atom[row_base + my_row] = ci;
    }
    __syncthreads();
    // fold K_l into c for pass 2 (D and the pass-1 staging are dead from here; their space
    // becomes the per-warp staging of pass 2)
    for (int e = tid; e < CT; e += kThreads) c_t[e] *= __ldg(p.kl + __ldg(p.l_of_lm + e % LM));

    // =========================== pass 2: the Jacobian rows ===========================
    const int NI = S * NCH;
    float4* wSD = reinterpret_cast<float4*>(smem + lay.w2 + wid * lay.w2_stride);         // [LM]
    float2* wG = reinterpret_cast<float2*>(smem + lay.w2 + wid * lay.w2_stride + 4 * LM);  // [NCH]
    float4* wUV = reinterpret_cast<float4*>(smem + lay.w2 + wid * lay.w2_stride + 4 * LM + ((2 * NCH + 3) & ~3));   // [NI]
    for (int g0 = 0; g0 < k_pairs; g0 += kGeoPairs) {
        const int gc = min(kGeoPairs, k_pairs - g0);
        __syncthreads();
        if (g0 > 0 || k_pairs > kGeoPairs) stage_geometry(g0, gc);     // otherwise still valid from pass 1
        __syncthreads();
        for (int pr = 0; pr < gc; ++pr) {
            const int4 gi = geo_i[pr];
            const int rw = gi.w;
            if (rw & kRowSelfImage) continue;
            const int row = rw & kRowMask;
            if ((row & (kWarps - 1)) != wid) continue;
            const bool accumulate = rw & kRowContinuation;
            const int Z = gi.z & 255;
            const float4 d = geo_d[pr];
            __syncwarp();
            // ---- radial factors and harmonics of this pair ----
            {
                const float t = __int_as_float(gi.y);
                const float rinv_h = p.inv_h / d.w;
                for (int ch = lane; ch < NCH; ch += 32) {
                    float v, dv;
                    radial_lookup(p.table, gi.x, NCH, ch, t, v, dv);
                    wG[ch] = make_float2(v, dv * rinv_h);
                }
                for (int t2 = lane; t2 < NQ; t2 += 32) {
                    const int lmp = __ldg(p.lm_of_t + t2);
                    const int l = lmp >> 4, m = lmp & 15;
                    float4 plus, minus;
                    solid_harmonic_item<L, true>(d.x, d.y, d.z, d.w * d.w, l, m, p.anorm, p.dfact, p.inv_int, plus, minus);
                    const int lm0 = l * l + l;
                    wSD[lm0 + m] = plus;
                    if (m) wSD[lm0 - m] = minus;
                }
            }
            __syncwarp();
            // ---- U, V for every (nu, n', l); items ordered l-major so that a warp's trip counts agree ----
            {
                const int SN = S * NMAX;
                for (int it = lane; it < NI; it += 32) {
                    const int l = it / SN, sn = it - l * SN;            // sn = nu * NMAX + n'
                    const float* cp = c_t + sn * LM + l * l;
                    const float4* hp = wSD + l * l;
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int m = 0; m <= 2 * l; ++m) {
                        const float cv = cp[m];
                        const float4 h = hp[m];
                        acc.x = fmaf(cv, h.x, acc.x); acc.y = fmaf(cv, h.y, acc.y);
                        acc.z = fmaf(cv, h.z, acc.z); acc.w = fmaf(cv, h.w, acc.w);
                    }
                    wUV[sn * L1 + l] = acc;                           // [nu][n'][l]
                }
            }
            __syncwarp();
            // ---- product rule and store ----
            float* out = p.out_jac + (size_t)(row_base + row) * 3 * F;
            if (!accumulate && lane == 0) p.row_atom[row_base + row] = key_atom(p.pair_key[pair_base + g0 + pr]);
            int boff = 0;
            for (int mu = 0; mu < S; ++mu) {
                for (int nu = mu; nu < S; ++nu) {
                    const int bsize = (mu == nu) ? (NMAX * (NMAX + 1) / 2) * L1 : NMAX * NCH;
                    float* ob = out + boff;
                    if (mu != Z && nu != Z) {
                        if (!accumulate)
                            for (int f = lane; f < bsize; f += 32) { ob[f] = 0.f; ob[F + f] = 0.f; ob[2 * F + f] = 0.f; }
                    } else if (mu == nu) {
                        // both terms; feature (n1 <= n2, l) sits at L1 (n1 NMAX - n1(n1-1)/2) + (n2-n1) L1 + l
                        const float4* UVz = wUV + Z * NCH;
                        for (int j = lane; j < NCH; j += 32) {
                            const int n2 = j / L1, l = j - n2 * L1;
                            const float2 gj = wG[j];
                            const float4 uj = UVz[j];
                            const float2* g1p = wG + l;
                            const float4* u1p = UVz + l;
                            float* o = ob + j;
                            for (int n1 = 0; n1 <= n2; ++n1) {
                                const float2 g1 = *g1p;
                                const float4 u1 = *u1p;
                                const float w = fmaf(g1.y, uj.x, gj.y * u1.x);    // Ghat_n1 U_n2 + Ghat_n2 U_n1
                                const float vx = fmaf(g1.x, uj.y, fmaf(gj.x, u1.y, w * d.x));
                                const float vy = fmaf(g1.x, uj.z, fmaf(gj.x, u1.z, w * d.y));
                                const float vz = fmaf(g1.x, uj.w, fmaf(gj.x, u1.w, w * d.z));
                                if (accumulate) { o[0] += vx; o[F] += vy; o[2 * F] += vz; }
                                else { o[0] = vx; o[F] = vy; o[2 * F] = vz; }
                                g1p += L1; u1p += L1;
                                o += (NMAX - n1 - 1) * L1;
                            }
                        }
                    } else if (mu == Z) {
                        // (grad c^mu_{n1 l}) c^nu_{n2 l}: G_{n1 l} V^nu_{n2 l} + Ghat_{n1 l} d U^nu_{n2 l}
                        for (int j = lane; j < NCH; j += 32) {
                            const int l = j % L1;
                            const float4 uj = wUV[nu * NCH + j];
                            const float xx = uj.x * d.x, xy = uj.x * d.y, xz = uj.x * d.z;
                            const float2* g1p = wG + l;
                            float* o = ob + j;
#pragma unroll 4
                            for (int n1 = 0; n1 < NMAX; ++n1) {
                                const float2 g1 = *g1p;
                                const float vx = fmaf(g1.x, uj.y, g1.y * xx);
                                const float vy = fmaf(g1.x, uj.z, g1.y * xy);
                                const float vz = fmaf(g1.x, uj.w, g1.y * xz);
                                if (accumulate) { o[0] += vx; o[F] += vy; o[2 * F] += vz; }
                                else { o[0] = vx; o[F] = vy; o[2 * F] = vz; }
                                g1p += L1; o += NCH;
                            }
                        }
                    } else {
                        // c^mu_{n1 l} (grad c^nu_{n2 l}): G_{n2 l} V^mu_{n1 l} + Ghat_{n2 l} d U^mu_{n1 l}
                        for (int j = lane; j < NCH; j += 32) {
                            const int l = j % L1;
                            const float2 gj = wG[j];
                            const float gx = gj.y * d.x, gy = gj.y * d.y, gz = gj.y * d.z;
                            const float4* u1p = wUV + mu * NCH + l;
                            float* o = ob + j;
#pragma unroll 4
                            for (int n1 = 0; n1 < NMAX; ++n1) {
                                const float4 u1 = *u1p;
                                const float vx = fmaf(gj.x, u1.y, gx * u1.x);
                                const float vy = fmaf(gj.x, u1.z, gy * u1.x);
                                const float vz = fmaf(gj.x, u1.w, gz * u1.x);
                                if (accumulate) { o[0] += vx; o[F] += vy; o[2 * F] += vz; }
                                else { o[0] = vx; o[F] = vy; o[2 * F] = vz; }
                                u1p += L1; o += NCH;
                            }
                        }
                    }
                    boff += bsize;
                }
            }
        }
    }
}

}  // namespace soap
