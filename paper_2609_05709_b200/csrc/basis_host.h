// Host-side construction of the radial tables and constants the kernels read.
// Built once per handle (construction is outside the timed region, as in the
// paper's Results section).  Plain C++ with libquadmath; no CUDA here.
#pragma once
#include <string>
#include <vector>

namespace soap {

constexpr int kTableDegree = 5;                    // per-interval polynomial degree
constexpr int kTableCoef = kTableDegree + 1;

struct HostBasis {
    int rbf = 0, n_max = 0, l_max = 0;
    double r_cut = 0, sigma = 0;
    int n_intervals = 0;                           // uniform intervals on [0, r_cut]
    double inv_h = 0;                              // n_intervals / r_cut
    // Radial factor G_nl(d) with c_nlm = sum_j G_nl(d_j) S_lm(d_j), S_lm the
    // real solid harmonic; table[(q * n_ch + n * (l_max+1) + l) * 6 + k] is the
    // coefficient of t^k on interval q, t = d * inv_h - q in [0, 1).
    std::vector<float> table;
    // the same functions on wider intervals (values only are read from it): descriptor-only kernel
    int n_intervals_values = 0;
    double inv_h_values = 0;
    std::vector<float> table_values;
    std::vector<float> self_term;                  // on-site c_n00, [n_max]
    std::vector<float> anorm;                      // harmonic normalisation, [(l,m), m<=l], sqrt2 folded in for m>0
    std::vector<float> dfact;                      // (2m-1)!!, [l_max+1]
    std::vector<float> kl;                         // pi sqrt(8/(2l+1)), [l_max+1]
};

// Returns 0 or a negative soap error code; `err` gets a message.
int build_basis(int rbf, double r_cut, int n_max, int l_max, double sigma,
                HostBasis& out, std::string& err);

// Evaluates the table in double precision at distance d: G[n_ch], Ghat[n_ch]
// (Ghat = (dG/dd)/d).  Used by the host-logic tests.
void eval_table(const HostBasis& b, double d, double* G, double* Ghat);

}  // namespace soap
