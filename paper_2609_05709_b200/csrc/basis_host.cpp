// Radial tables and constants, computed on the host in quad precision.
//
// Both radial families of the paper reduce to one radial factor per pair,
//   c^mu_nlm = sum_j G_nl(d_j) S_lm(d_j),   S_lm = r^l Y_lm (real solid harmonic),
// with
//   Gaussian-type orbitals (Eq. 13):
//     G_nl(d) = (2 pi)^(3/2) sigma^3 sum_k beta^l_nk (1 + 2 sigma^2 alpha_kl)^-(l+3/2)
//               exp(-alpha_kl d^2 / (1 + 2 sigma^2 alpha_kl)),
//   polynomials (Eqs. 18-19, divided by d^l):
//     G_nl(d) = 4 pi int_0^rcut r^2 g_n(r) exp(-(r-d)^2 / 2 sigma^2) (r/sigma^2)^l
//               [exp(-z) i_l(z) / z^l] dr,   z = r d / sigma^2.
// The Loewdin matrices (Eq. 9, and W = S^(-1/2) below Eq. 17) are so
// ill-conditioned that a fp32 (or even fp64) evaluation of the k-sum loses the
// result; here the sums are done once in __float128 and the smooth, O(1)
// functions G_nl(d) are stored as degree-5 polynomials on uniform intervals of
// d, which the kernels evaluate in fp32 without cancellation.  dG/dd comes
// from the same polynomial.
#include "basis_host.h"

#include <quadmath.h>

#include <algorithm>
#include <cmath>
#include <cstdio>

#include "soap.h"

namespace soap {
namespace {

typedef __float128 quad;
typedef long double ld;

// Cyclic Jacobi for a symmetric positive-definite matrix; the off-diagonal test
// is relative to sqrt(a_pp a_qq), which keeps the small eigenvalues accurate.
void jacobi_eigen(int n, std::vector<quad>& A, std::vector<quad>& V) {
    V.assign(n * n, 0);
    for (int i = 0; i < n; ++i) V[i * n + i] = 1;
    const quad eps = 1e-33Q;
    for (int sweep = 0; sweep < 200; ++sweep) {
        bool rotated = false;
        for (int p = 0; p < n - 1; ++p) {
            for (int q = p + 1; q < n; ++q) {
                quad apq = A[p * n + q];
                if (fabsq(apq) <= eps * sqrtq(fabsq(A[p * n + p] * A[q * n + q]))) continue;
                rotated = true;
                quad theta = (A[q * n + q] - A[p * n + p]) / (2 * apq);
                quad t = (theta >= 0 ? 1 : -1) / (fabsq(theta) + sqrtq(theta * theta + 1));
                quad c = 1 / sqrtq(t * t + 1), s = t * c;
                for (int k = 0; k < n; ++k) {           // columns p, q
                    quad akp = A[k * n + p], akq = A[k * n + q];
                    A[k * n + p] = c * akp - s * akq;
                    A[k * n + q] = s * akp + c * akq;
                }
                for (int k = 0; k < n; ++k) {           // rows p, q
                    quad apk = A[p * n + k], aqk = A[q * n + k];
                    A[p * n + k] = c * apk - s * aqk;
                    A[q * n + k] = s * apk + c * aqk;
                }
                for (int k = 0; k < n; ++k) {
                    quad vkp = V[k * n + p], vkq = V[k * n + q];
                    V[k * n + p] = c * vkp - s * vkq;
                    V[k * n + q] = s * vkp + c * vkq;
                }
            }
        }
        if (!rotated) break;
    }
}

// Principal inverse square root of a symmetric positive-definite matrix.
bool inv_sqrt_spd(int n, const std::vector<quad>& S, std::vector<quad>& out) {
    std::vector<quad> A = S, V;
    jacobi_eigen(n, A, V);
    out.assign(n * n, 0);
    for (int k = 0; k < n; ++k)
        if (!(A[k * n + k] > 0)) return false;
    for (int a = 0; a < n; ++a)
        for (int b = 0; b < n; ++b) {
            quad acc = 0;
            for (int k = 0; k < n; ++k) acc += V[a * n + k] * V[b * n + k] / sqrtq(A[k * n + k]);
            out[a * n + b] = acc;
        }
    return true;
}

// Inverse of the 6x6 Vandermonde matrix of the Chebyshev nodes on (0, 1).
void vandermonde_inverse(quad nodes[kTableCoef], quad inv[kTableCoef][kTableCoef]) {
    const int m = kTableCoef;
    quad a[m][2 * m];
    for (int k = 0; k < m; ++k) {
        nodes[k] = (1 - cosq(M_PIq * (k + 0.5Q) / m)) / 2;
        quad p = 1;
        for (int j = 0; j < m; ++j) { a[k][j] = p; p *= nodes[k]; }
        for (int j = 0; j < m; ++j) a[k][m + j] = (j == k) ? 1 : 0;
    }
    for (int c = 0; c < m; ++c) {
        int piv = c;
        for (int r = c + 1; r < m; ++r) if (fabsq(a[r][c]) > fabsq(a[piv][c])) piv = r;
        for (int j = 0; j < 2 * m; ++j) std::swap(a[c][j], a[piv][j]);
        quad d = a[c][c];
        for (int j = 0; j < 2 * m; ++j) a[c][j] /= d;
        for (int r = 0; r < m; ++r) {
            if (r == c) continue;
            quad f = a[r][c];
            for (int j = 0; j < 2 * m; ++j) a[r][j] -= f * a[c][j];
        }
    }
    for (int i = 0; i < m; ++i) for (int j = 0; j < m; ++j) inv[i][j] = a[i][m + j];
}

// G_nl at a list of distances, Gaussian-type orbitals.  out[(i * n_ch) + n*(L+1)+l].
void gto_values(double r_cut, int n_max, int l_max, double sigma,
                const std::vector<quad>& d, std::vector<quad>& out) {
    const int L1 = l_max + 1, n_ch = n_max * L1;
    out.assign(d.size() * n_ch, 0);
    const quad s2 = (quad)sigma * (quad)sigma;
    const quad pref = powq(2 * M_PIq, 1.5Q) * (quad)sigma * s2;
    for (int l = 0; l < L1; ++l) {
        std::vector<quad> alpha(n_max), S(n_max * n_max), beta;
        for (int k = 0; k < n_max; ++k) {
            // Eq. 10; a lone primitive sits at z = 1
            quad z = (n_max == 1) ? 1 : 1 + (quad)k * ((quad)r_cut - 1) / (n_max - 1);
            alpha[k] = (3 * logq(10.0Q) + l * logq(z)) / (z * z);
        }
        const quad gam = tgammaq(l + 1.5Q);
        for (int a = 0; a < n_max; ++a)                      // Eq. 8
            for (int b = 0; b < n_max; ++b)
                S[a * n_max + b] = gam / (2 * powq(alpha[a] + alpha[b], l + 1.5Q));
        inv_sqrt_spd(n_max, S, beta);                        // Eq. 9
        std::vector<quad> amp(n_max), ak(n_max);
        for (int k = 0; k < n_max; ++k) {
            quad w = 1 + 2 * s2 * alpha[k];
            amp[k] = pref * powq(w, -(l + 1.5Q));
            ak[k] = alpha[k] / w;
        }
        std::vector<quad> prim(n_max);
        for (size_t i = 0; i < d.size(); ++i) {
            for (int k = 0; k < n_max; ++k) prim[k] = amp[k] * expq(-ak[k] * d[i] * d[i]);
            for (int n = 0; n < n_max; ++n) {
                quad acc = 0;
                for (int k = 0; k < n_max; ++k) acc += beta[n * n_max + k] * prim[k];
                out[i * n_ch + n * L1 + l] = acc;
            }
        }
    }
}

// Gauss-Legendre nodes and weights on [-1, 1] by Newton iteration.
void gauss_legendre(int n, std::vector<ld>& x, std::vector<ld>& w) {
    x.resize(n); w.resize(n);
    for (int i = 0; i < n; ++i) {
        ld z = cosl(M_PIl * (i + 0.75L) / (n + 0.5L)), pp = 0;
        for (int it = 0; it < 100; ++it) {
            ld p1 = 1, p2 = 0;
            for (int j = 1; j <= n; ++j) { ld p3 = p2; p2 = p1; p1 = ((2 * j - 1) * z * p2 - (j - 1) * p3) / j; }
            pp = n * (z * p1 - p2) / (z * z - 1);
            ld dz = p1 / pp;
            z -= dz;
            if (fabsl(dz) < 1e-19L) break;
        }
        x[i] = z; w[i] = 2 / ((1 - z * z) * pp * pp);
    }
}

// T_l(z) = i_l(z) / z^l for l = 0..L (modified spherical Bessel function of
// the first kind).  Power series for the two highest orders (all terms
// positive), then the downward recurrence T_{l-1} = z^2 T_{l+1} + (2l+1) T_l.
void bessel_i_over_zl(int L, ld z, ld* T) {
    auto series = [&](int l) {
        ld dfact = 1;
        for (int j = 1; j <= l; ++j) dfact *= (2 * j + 1);            // (2l+1)!!
        ld term = 1 / dfact, sum = term, h = z * z / 2;
        for (int k = 1; k < 100000; ++k) {
            term *= h / ((ld)k * (2 * l + 2 * k + 1));
            sum += term;
            if (term < sum * 1e-22L) break;
        }
        return sum;
    };
    T[L] = series(L);
    if (L >= 1) T[L - 1] = series(L - 1);
    for (int l = L - 1; l >= 1; --l) T[l - 1] = z * z * T[l + 1] + (2 * l + 1) * T[l];
}

// G_nl at a list of distances, polynomial basis.
bool poly_values(double r_cut, int n_max, int l_max, double sigma,
                 const std::vector<quad>& d, std::vector<quad>& out) {
    const int L1 = l_max + 1, n_ch = n_max * L1;
    out.assign(d.size() * n_ch, 0);
    // W = S^(-1/2), Eq. 17 (k = 1..n_max)
    std::vector<quad> S(n_max * n_max), W;
    for (int a = 1; a <= n_max; ++a)
        for (int b = 1; b <= n_max; ++b)
            S[(a - 1) * n_max + (b - 1)] = sqrtq((quad)((5 + 2 * a) * (5 + 2 * b))) / (5 + a + b);
    if (!inv_sqrt_spd(n_max, S, W)) return false;
    // composite Gauss-Legendre on [0, r_cut]: panels about sigma/2 wide, 16 nodes each
    const int per = 16;
    int panels = std::max(8, (int)std::ceil(r_cut / (0.5 * sigma)));
    std::vector<ld> gx, gw;
    gauss_legendre(per, gx, gw);
    const int nq = panels * per;
    std::vector<ld> r(nq), w(nq);
    for (int p = 0; p < panels; ++p)
        for (int i = 0; i < per; ++i) {
            ld a = (ld)r_cut * p / panels, b = (ld)r_cut * (p + 1) / panels;
            r[p * per + i] = (a + b) / 2 + (b - a) / 2 * gx[i];
            w[p * per + i] = (b - a) / 2 * gw[i];
        }
    // orthonormal radial functions g_n(r_q), Eq. 15, k-sum in quad
    std::vector<ld> g(n_max * nq);
    for (int qi = 0; qi < nq; ++qi) {
        std::vector<quad> prim(n_max);
        quad x = (quad)r_cut - (quad)r[qi];
        for (int k = 1; k <= n_max; ++k) {
            quad Nk = sqrtq(powq((quad)r_cut, 2 * k + 5) / (2 * k + 5));   // Eq. 16
            prim[k - 1] = powq(x, k + 2) / Nk;
        }
        for (int n = 0; n < n_max; ++n) {
            quad acc = 0;
            for (int k = 0; k < n_max; ++k) acc += W[n * n_max + k] * prim[k];
            g[n * nq + qi] = (ld)acc;
        }
    }
    const ld s2 = (ld)sigma * (ld)sigma;
    std::vector<ld> T(L1), acc(n_ch);
    for (size_t i = 0; i < d.size(); ++i) {
        ld di = (ld)d[i];
        std::fill(acc.begin(), acc.end(), 0.0L);
        for (int qi = 0; qi < nq; ++qi) {
            ld dr = r[qi] - di;
            if (dr * dr > 2 * s2 * 90.0L) continue;                     // exp(-90) ~ 1e-39
            ld z = r[qi] * di / s2;
            bessel_i_over_zl(l_max, z, T.data());
            ld base = w[qi] * r[qi] * r[qi] * expl(-dr * dr / (2 * s2) - z);
            ld rl = 1;                                                  // (r / sigma^2)^l
            for (int l = 0; l < L1; ++l) {
                ld f = base * rl * T[l];
                for (int n = 0; n < n_max; ++n) acc[n * L1 + l] += g[n * nq + qi] * f;
                rl *= r[qi] / s2;
            }
        }
        for (int c = 0; c < n_ch; ++c) out[i * n_ch + c] = 4 * M_PIq * (quad)acc[c];
    }
    return true;
}

}  // namespace

int build_basis(int rbf, double r_cut, int n_max, int l_max, double sigma,
                HostBasis& out, std::string& err) {
    if (!(r_cut > 0) || !(sigma > 0) || n_max < 1 || n_max > 16 || l_max < 0 || l_max > 12) {
        err = "need r_cut > 0, sigma > 0, 1 <= n_max <= 16, 0 <= l_max <= 12";
        return SOAP_ERR_INVALID_ARG;
    }
    if (rbf != 0 && rbf != 1) { err = "rbf must be 0 (GTO) or 1 (polynomial)"; return SOAP_ERR_INVALID_ARG; }
    if (rbf == 0 && !(r_cut > 1.0)) {
        err = "the GTO width rule (Eq. 10) places primitives between 1 A and r_cut: need r_cut > 1";
        return SOAP_ERR_INVALID_ARG;
    }
    out = HostBasis();
    out.rbf = rbf; out.n_max = n_max; out.l_max = l_max; out.r_cut = r_cut; out.sigma = sigma;
    const int L1 = l_max + 1, n_ch = n_max * L1;
    quad nodes[kTableCoef], vinv[kTableCoef][kTableCoef];
    vandermonde_inverse(nodes, vinv);
    std::vector<quad> vals;
    // Fits the per-interval polynomials on `nint` uniform intervals; `vals` keeps the samples, the last of
    // which is the value at distance zero.
    auto fit = [&](int nint, std::vector<float>& table) -> bool {
        const quad inv_h = (quad)nint / (quad)r_cut;
        std::vector<quad> d((size_t)nint * kTableCoef + 1);
        for (int q = 0; q < nint; ++q)
            for (int k = 0; k < kTableCoef; ++k)
                d[(size_t)q * kTableCoef + k] = ((quad)q + nodes[k]) / inv_h;
        d.back() = 0;                                               // for the on-site term
        if (rbf == 0) gto_values(r_cut, n_max, l_max, sigma, d, vals);
        else if (!poly_values(r_cut, n_max, l_max, sigma, d, vals)) return false;
        table.resize((size_t)nint * n_ch * kTableCoef);
        for (int q = 0; q < nint; ++q)
            for (int c = 0; c < n_ch; ++c)
                for (int j = 0; j < kTableCoef; ++j) {
                    quad acc = 0;
                    for (int k = 0; k < kTableCoef; ++k)
                        acc += vinv[j][k] * vals[((size_t)q * kTableCoef + k) * n_ch + c];
                    table[((size_t)q * n_ch + c) * kTableCoef + j] = (float)acc;
                }
        return true;
    };
    // The descriptor-only kernel keeps its table in shared memory and reads values only: on intervals of sigma/4
    // the degree-5 fit error (1e-8 of a channel's maximum) still sits below the fp32 rounding of the coefficients
    // (5e-8), at two thirds of the size; sigma/3 would be smaller still but loses accuracy in the tails, where
    // the functions are small.
    int nint_v = (int)std::ceil(r_cut / (sigma / 4.0));
    nint_v = std::min(std::max(nint_v, 8), 4096);
    out.n_intervals_values = nint_v;
    out.inv_h_values = nint_v / r_cut;
    if (!fit(nint_v, out.table_values)) {
        err = "polynomial overlap matrix is not positive definite at this n_max";
        return SOAP_ERR_INVALID_ARG;
    }
    // interval width about sigma/6: the degree-5 fit (value and derivative) then sits at the fp32 rounding floor
    int nint = (int)std::ceil(r_cut / (sigma / 6.0));
    nint = std::min(std::max(nint, 16), 4096);
    out.n_intervals = nint;
    out.inv_h = nint / r_cut;
    if (!fit(nint, out.table)) {
        err = "polynomial overlap matrix is not positive definite at this n_max";
        return SOAP_ERR_INVALID_ARG;
    }
    // on-site term: a neighbour at distance zero, S_00 = 1/sqrt(4 pi)   (second term of Eq. 13)
    out.self_term.resize(n_max);
    for (int n = 0; n < n_max; ++n)
        out.self_term[n] = (float)(vals[(size_t)nint * kTableCoef * n_ch + n * L1] / sqrtq(4 * M_PIq));
    // harmonic normalisation sqrt((2l+1)/4pi (l-m)!/(l+m)!), times sqrt2 for m > 0
    out.anorm.resize(L1 * (L1 + 1) / 2);
    for (int l = 0; l < L1; ++l)
        for (int m = 0; m <= l; ++m) {
            quad ratio = 1;
            for (int j = l - m + 1; j <= l + m; ++j) ratio /= j;
            quad a = sqrtq((2 * l + 1) / (4 * M_PIq) * ratio);
            if (m > 0) a *= sqrtq(2.0Q);
            out.anorm[l * (l + 1) / 2 + m] = (float)a;
        }
    out.dfact.resize(L1);
    quad df = 1;
    for (int m = 0; m < L1; ++m) { if (m > 0) df *= (2 * m - 1); out.dfact[m] = (float)df; }
    out.kl.resize(L1);
    for (int l = 0; l < L1; ++l) out.kl[l] = (float)(M_PIq * sqrtq(8.0Q / (2 * l + 1)));   // prefactor of Eq. 4
    return 0;
}

void eval_table(const HostBasis& b, double d, double* G, double* Ghat) {
    const int n_ch = b.n_max * (b.l_max + 1);
    double u = d * b.inv_h;
    int q = std::min(std::max((int)u, 0), b.n_intervals - 1);
    double t = u - q;
    for (int c = 0; c < n_ch; ++c) {
        const float* p = &b.table[((size_t)q * n_ch + c) * kTableCoef];
        double v = 0, dv = 0;
        for (int k = kTableDegree; k >= 0; --k) {
            dv = dv * t + v;
            v = v * t + p[k];
        }
        G[c] = v;
        Ghat[c] = d > 0 ? dv * b.inv_h / d : 0.0;
    }
}

}  // namespace soap
