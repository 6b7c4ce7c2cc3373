// The fused per-centre kernel: one CTA owns one centre atom and produces its
// descriptor row (Eq. 4) and, in the derivative build, all of its Jacobian
// rows (Eq. 5).  Nothing per pair ever goes to HBM: radial factors, solid
// harmonics and the precontracted U/V live in shared memory for a chunk of
// pairs at a time; the expansion coefficients c^mu_nlm of the centre stay in
// shared memory for the whole CTA lifetime.
//
// Per pair (displacement d = r_j + T - r_i, species Z of j):
//   c^Z_nlm        += G_nl(|d|) S_lm(d)                               (Eq. 13 / 18)
//   grad_j c^Z_nlm  = G_nl grad S_lm + Ghat_nl d S_lm,  Ghat = G'/|d|  (Eq. 14 / 23)
// with S_lm = r^l Y_lm the real solid harmonic and G_nl, G'_nl read from the
// degree-5 tables.  Pass 1 accumulates c and D = sum_j grad_j c (for the
// centre's own row, which is minus the sum over the neighbours).  Pass 2 forms,
// per pair, U^nu_{n'l} = K_l sum_m S_lm c^nu_{n'lm} and V likewise with grad S,
// and then each output element of Eq. 5 is two fused multiply-adds per term.
#pragma once
#include "soap_device.cuh"

namespace soap {

__device__ inline int tri_index(int l, int m) { return l * (l + 1) / 2 + m; }

template <bool DERIV>
__global__ void __launch_bounds__(kThreads)
center_kernel(const CenterParams p) {
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const long long c_idx = blockIdx.x;
    // a failed neighbour build or an undersized output: write nothing
    if (p.pair_ptr[p.n_centers] > p.pair_capacity) return;
    if (DERIV && p.row_ptr[p.n_centers] > p.row_capacity) {
        if (c_idx == 0 && tid == 0) atomicOr(&p.counters->status, kStatusRowCapacity);
        return;
    }
    const int S = p.S, NMAX = p.n_max, L = p.l_max, L1 = L + 1, LM = L1 * L1, NCH = NMAX * L1;
    const int NE = NMAX * LM, CT = S * NE, NQ = L1 * (L1 + 1) / 2, P = p.P, F = p.F;
    const SmemLayout lay = make_layout(S, NMAX, L, P, DERIV);
    float* c_t = smem + lay.c;
    float* D_t = smem + lay.D;                             // [3][CT]
    float4* sd = reinterpret_cast<float4*>(smem + lay.sd); // dx, dy, dz, r
    int2* sinfo = reinterpret_cast<int2*>(smem + lay.sinfo);   // species | moving<<8 ; pair_row word
    float* sS = smem + lay.sSD;                            // desc: [P][LM]
    float4* sSD4 = reinterpret_cast<float4*>(smem + lay.sSD);  // deriv: [P][LM] (S, dSx, dSy, dSz)
    float* sG1 = smem + lay.sG;                            // desc: [P][NCH]
    float2* sG2 = reinterpret_cast<float2*>(smem + lay.sG);    // deriv: [P][NCH] (G, Ghat)
    float* sQ = smem + lay.sQ;                             // [P][NQ]
    float2* sCS = reinterpret_cast<float2*>(smem + lay.sCS);   // [P][L1]
    float4* sUV = reinterpret_cast<float4*>(smem + lay.sUV);   // [P][S*NCH]

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
    int el_lm[kMaxElemPerThread], el_ch[kMaxElemPerThread];
#pragma unroll
    for (int k = 0; k < kMaxElemPerThread; ++k) {
        int e = tid + k * kThreads;
        int n = e / LM, lm = e - n * LM;
        int l = (int)sqrtf((float)lm);
        while ((l + 1) * (l + 1) <= lm) ++l;
        while (l * l > lm) --l;
        el_lm[k] = e < NE ? lm : -1;
        el_ch[k] = n * L1 + l;
    }

    // ---- stage one chunk of pairs: geometry, radial factors, solid harmonics ----
    auto stage_chunk = [&](int q0, int pc) {
        if (tid < pc) {
            const unsigned long long key = p.pair_key[pair_base + q0 + tid];
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
            sd[tid] = make_float4((float)dx, (float)dy, (float)dz, (float)r);
            const int rw = p.pair_row[pair_base + q0 + tid];
            sinfo[tid] = make_int2(p.species_idx[j] | ((rw & kRowSelfImage) ? 0 : 256), rw);
            // interval and offset in the radial table, in fp64 so that the offset keeps its digits
            double u = r * (double)p.inv_h;
            int qi = min((int)u, p.n_intervals - 1);
            sCS[tid * L1] = make_float2(__int_as_float(qi), (float)(u - qi));   // parked here until the harmonics overwrite it
        }
        __syncthreads();
        // radial factors: thread <-> (pair, channel)
        for (int idx = tid; idx < pc * NCH; idx += kThreads) {
            const int pr = idx / NCH, ch = idx - pr * NCH;
            const float2 it = sCS[pr * L1];
            const int qi = __float_as_int(it.x);
            const float t = it.y;
            const float2* cf = reinterpret_cast<const float2*>(p.table + ((size_t)qi * NCH + ch) * 6);
            const float2 a = __ldg(cf), b = __ldg(cf + 1), cc = __ldg(cf + 2);
            float v = cc.y, dv = 0.f;
            dv = fmaf(dv, t, v); v = fmaf(v, t, cc.x);
            dv = fmaf(dv, t, v); v = fmaf(v, t, b.y);
            dv = fmaf(dv, t, v); v = fmaf(v, t, b.x);
            dv = fmaf(dv, t, v); v = fmaf(v, t, a.y);
            dv = fmaf(dv, t, v); v = fmaf(v, t, a.x);
            if (DERIV) sG2[pr * NCH + ch] = make_float2(v, dv * p.inv_h / sd[pr].w);
            else sG1[pr * NCH + ch] = v;
        }
        __syncthreads();
        // harmonics, step 1: thread <-> (pair, m): (x+iy)^m and the column Q_l^m, l = m..L
        for (int idx = tid; idx < pc * L1; idx += kThreads) {
            const int pr = idx / L1, m = idx - pr * L1;
            const float4 d = sd[pr];
            float cm = 1.f, sm = 0.f;
            for (int t = 0; t < m; ++t) {
                const float cn = d.x * cm - d.y * sm;
                sm = d.x * sm + d.y * cm;
                cm = cn;
            }
            sCS[pr * L1 + m] = make_float2(cm, sm);
            const float r2 = d.w * d.w;
            float q0v = 0.f, q1v = __ldg(p.dfact + m);          // Q_m^m = (2m-1)!!
            sQ[pr * NQ + tri_index(m, m)] = q1v;
            for (int l = m + 1; l <= L; ++l) {
                // (l-m) Q_l^m = (2l-1) z Q_{l-1}^m - (l+m-1) r^2 Q_{l-2}^m
                const float qn = ((2 * l - 1) * d.z * q1v - (l + m - 1) * r2 * q0v) / (float)(l - m);
                q0v = q1v; q1v = qn;
                sQ[pr * NQ + tri_index(l, m)] = qn;
            }
        }
        __syncthreads();
        // harmonics, step 2: thread <-> (pair, l, m >= 0): S_{l,+-m} and, for the Jacobian, their gradients
        for (int idx = tid; idx < pc * NQ; idx += kThreads) {
            const int pr = idx / NQ, t = idx - pr * NQ;
            int l = (int)((sqrtf(8.f * t + 1.f) - 1.f) * 0.5f);
            while (tri_index(l + 1, 0) <= t) ++l;
            while (tri_index(l, 0) > t) --l;
            const int m = t - tri_index(l, 0);
            const float a = __ldg(p.anorm + t);
            const float Q = sQ[pr * NQ + t];
            const float2 cs = sCS[pr * L1 + m];
            const int lm0 = l * l + l;
            if (!DERIV) {
                if (m == 0) sS[pr * LM + lm0] = a * Q;
                else { sS[pr * LM + lm0 + m] = a * Q * cs.x; sS[pr * LM + lm0 - m] = a * Q * cs.y; }
            } else {
                const float4 d = sd[pr];
                // dQ_l^m/dx = -x Q_{l-1}^{m+1}, dQ_l^m/dy = -y Q_{l-1}^{m+1}, dQ_l^m/dz = (l+m) Q_{l-1}^m
                const float Qx = (l - 1 >= m + 1) ? sQ[pr * NQ + tri_index(l - 1, m + 1)] : 0.f;
                const float Qz = (l - 1 >= m) ? (l + m) * sQ[pr * NQ + tri_index(l - 1, m)] : 0.f;
                if (m == 0) {
                    sSD4[pr * LM + lm0] = make_float4(a * Q, -a * d.x * Qx, -a * d.y * Qx, a * Qz);
                } else {
                    const float2 cp = sCS[pr * L1 + m - 1];
                    const float mq = m * Q;
                    // d/dx (x+iy)^m = m (x+iy)^(m-1), d/dy = i m (x+iy)^(m-1)
                    sSD4[pr * LM + lm0 + m] = make_float4(a * Q * cs.x, a * (-d.x * Qx * cs.x + mq * cp.x),
                                                         a * (-d.y * Qx * cs.x - mq * cp.y), a * Qz * cs.x);
                    sSD4[pr * LM + lm0 - m] = make_float4(a * Q * cs.y, a * (-d.x * Qx * cs.y + mq * cp.y),
                                                         a * (-d.y * Qx * cs.y + mq * cp.x), a * Qz * cs.y);
                }
            }
        }
        __syncthreads();
    };

    // =========================== pass 1: c (and D) ===========================
    for (int q0 = 0; q0 < k_pairs; q0 += P) {
        const int pc = min(P, k_pairs - q0);
        stage_chunk(q0, pc);
        for (int s = 0; s < S; ++s) {
            float ac[kMaxElemPerThread], ax[kMaxElemPerThread], ay[kMaxElemPerThread], az[kMaxElemPerThread];
#pragma unroll
            for (int k = 0; k < kMaxElemPerThread; ++k) ac[k] = ax[k] = ay[k] = az[k] = 0.f;
            bool any = false;
            for (int pr = 0; pr < pc; ++pr) {
                const int info = sinfo[pr].x;
                if ((info & 255) != s) continue;
                any = true;
                if (!DERIV) {
#pragma unroll
                    for (int k = 0; k < kMaxElemPerThread; ++k)
                        if (el_lm[k] >= 0) ac[k] = fmaf(sG1[pr * NCH + el_ch[k]], sS[pr * LM + el_lm[k]], ac[k]);
                } else {
                    const float4 d = sd[pr];
                    const float mv = (info & 256) ? 1.f : 0.f;   // an image of the centre does not move relative to it
#pragma unroll
                    for (int k = 0; k < kMaxElemPerThread; ++k)
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
                for (int k = 0; k < kMaxElemPerThread; ++k)
                    if (el_lm[k] >= 0) {
                        const int e = s * NE + tid + k * kThreads;
                        c_t[e] += ac[k];
                        if (DERIV) { D_t[e] += ax[k]; D_t[CT + e] += ay[k]; D_t[2 * CT + e] += az[k]; }
                    }
            }
        }
        __syncthreads();
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
            for (int dir = 0; dir < 3; ++dir) {
                const float* Da = D_t + dir * CT + ia;
                const float* Db = D_t + dir * CT + ib;
                float acc = 0.f;
                for (int m = 0; m <= 2 * l; ++m) acc = fmaf(Da[m], c_t[ib + m], fmaf(c_t[ia + m], Db[m], acc));
                out[(size_t)dir * F + f] = kl * acc;
            }
        }
        if (tid == 0) p.row_atom[row_base + my_row] = ci;
    }
    __syncthreads();
    // fold K_l into c for pass 2 (D is dead from here; its space becomes the U/V staging)
    for (int e = tid; e < CT; e += kThreads) {
        int lm = e % LM;
        int l = (int)sqrtf((float)lm);
        while ((l + 1) * (l + 1) <= lm) ++l;
        while (l * l > lm) --l;
        c_t[e] *= __ldg(p.kl + l);
    }
    __syncthreads();

    // lane-fixed channels j = (n', l) of phase C
    const int NI = S * NCH;
    // =========================== pass 2: the Jacobian rows ===========================
    for (int q0 = 0; q0 < k_pairs; q0 += P) {
        const int pc = min(P, k_pairs - q0);
        stage_chunk(q0, pc);
        // ---- phase B: U, V per pair and (nu, n', l); a thread serves 4 pairs of one item ----
        const int groups = (pc + 3) >> 2;
        for (int unit = tid; unit < groups * NI; unit += kThreads) {
            const int pg = unit / NI, item = unit - pg * NI;
            const int l = item % L1;
            const float* cp = c_t + (item / L1) * LM + l * l;
            float4 acc[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) acc[a] = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int m = 0; m <= 2 * l; ++m) {
                const float cv = cp[m];
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    const float4 h = sSD4[(pg * 4 + a) * LM + l * l + m];
                    acc[a].x = fmaf(cv, h.x, acc[a].x);
                    acc[a].y = fmaf(cv, h.y, acc[a].y);
                    acc[a].z = fmaf(cv, h.z, acc[a].z);
                    acc[a].w = fmaf(cv, h.w, acc[a].w);
                }
            }
#pragma unroll
            for (int a = 0; a < 4; ++a) sUV[(pg * 4 + a) * NI + item] = acc[a];
        }
        __syncthreads();
        // ---- phase C: product rule and store; a warp owns whole rows ----
        for (int pr = 0; pr < pc; ++pr) {
            const int2 info = sinfo[pr];
            const int rw = info.y;
            if (rw & kRowSelfImage) continue;
            const int row = rw & kRowMask;
            if ((row % kWarps) != wid) continue;
            const bool accumulate = rw & kRowContinuation;
            const int Z = info.x & 255;
            const float4 d = sd[pr];
            float* out = p.out_jac + (size_t)(row_base + row) * 3 * F;
            if (!accumulate && lane == 0) p.row_atom[row_base + row] = key_atom(p.pair_key[pair_base + q0 + pr]);
            const float2* G = sG2 + pr * NCH;
            const float4* UV = sUV + pr * NI;
            int boff = 0;
            for (int mu = 0; mu < S; ++mu) {
                for (int nu = mu; nu < S; ++nu) {
                    const int bsize = (mu == nu) ? (NMAX * (NMAX + 1) / 2) * L1 : NMAX * NCH;
                    float* ob = out + boff;
                    if (mu != Z && nu != Z) {
                        if (!accumulate)
                            for (int f = lane; f < bsize; f += 32) { ob[f] = 0.f; ob[F + f] = 0.f; ob[2 * F + f] = 0.f; }
                    } else if (mu == nu) {
                        // both terms; features (n1 <= n2, l) at tri(n1) + (n2-n1) L1 + l
                        for (int j = lane; j < NCH; j += 32) {
                            const int n2 = j / L1, l = j - n2 * L1;
                            const float2 gj = G[j];
                            const float4 uj = UV[Z * NCH + j];
                            const float tj = gj.y;
                            for (int n1 = 0; n1 <= n2; ++n1) {
                                const int i1 = n1 * L1 + l;
                                const float2 g1 = G[i1];
                                const float4 u1 = UV[Z * NCH + i1];
                                const float w = g1.y * uj.x + tj * u1.x;          // Ghat_n1 U_n2 + Ghat_n2 U_n1
                                const float vx = fmaf(g1.x, uj.y, fmaf(gj.x, u1.y, w * d.x));
                                const float vy = fmaf(g1.x, uj.z, fmaf(gj.x, u1.z, w * d.y));
                                const float vz = fmaf(g1.x, uj.w, fmaf(gj.x, u1.w, w * d.z));
                                const int f = (n1 * NMAX - n1 * (n1 - 1) / 2) * L1 + (n2 - n1) * L1 + l;
                                if (accumulate) { ob[f] += vx; ob[F + f] += vy; ob[2 * F + f] += vz; }
                                else { ob[f] = vx; ob[F + f] = vy; ob[2 * F + f] = vz; }
                            }
                        }
                    } else if (mu == Z) {
                        // (grad c^mu_{n1 l}) c^nu_{n2 l}: G_{n1 l} V^nu_{n2 l} + Ghat_{n1 l} d U^nu_{n2 l}
                        for (int j = lane; j < NCH; j += 32) {
                            const int l = j % L1;
                            const float4 uj = UV[nu * NCH + j];
                            const float xx = uj.x * d.x, xy = uj.x * d.y, xz = uj.x * d.z;
                            for (int n1 = 0; n1 < NMAX; ++n1) {
                                const float2 g1 = G[n1 * L1 + l];
                                const float vx = fmaf(g1.x, uj.y, g1.y * xx);
                                const float vy = fmaf(g1.x, uj.z, g1.y * xy);
                                const float vz = fmaf(g1.x, uj.w, g1.y * xz);
                                const int f = n1 * NCH + j;
                                if (accumulate) { ob[f] += vx; ob[F + f] += vy; ob[2 * F + f] += vz; }
                                else { ob[f] = vx; ob[F + f] = vy; ob[2 * F + f] = vz; }
                            }
                        }
                    } else {
                        // c^mu_{n1 l} (grad c^nu_{n2 l}): G_{n2 l} V^mu_{n1 l} + Ghat_{n2 l} d U^mu_{n1 l}
                        for (int j = lane; j < NCH; j += 32) {
                            const int l = j % L1;
                            const float2 gj = G[j];
                            const float gx = gj.y * d.x, gy = gj.y * d.y, gz = gj.y * d.z;
                            for (int n1 = 0; n1 < NMAX; ++n1) {
                                const float4 u1 = UV[mu * NCH + n1 * L1 + l];
                                const float vx = fmaf(gj.x, u1.y, gx * u1.x);
                                const float vy = fmaf(gj.x, u1.z, gy * u1.x);
                                const float vz = fmaf(gj.x, u1.w, gz * u1.x);
                                const int f = n1 * NCH + j;
                                if (accumulate) { ob[f] += vx; ob[F + f] += vy; ob[2 * F + f] += vz; }
                                else { ob[f] = vx; ob[F + f] = vy; ob[2 * F + f] = vz; }
                            }
                        }
                    }
                    boff += bsize;
                }
            }
        }
        __syncthreads();
    }
}

}  // namespace soap
