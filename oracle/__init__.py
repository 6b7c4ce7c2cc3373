"""fp64 CPU oracle for the SOAP hot path.  TEST INFRASTRUCTURE ONLY.

This package is the yardstick the CUDA library is measured against.  It is a
plain, slow NumPy restatement of what the paper defines: Gaussian-smeared
species densities (Eq. 1) projected on radial functions times real spherical
harmonics (Eq. 3), contracted to the partial power spectrum (Eq. 4) and
differentiated by the product rule (Eq. 5), with the Gaussian-type-orbital
basis of Eqs. 6-10 and 13-14 and the polynomial basis of Eqs. 15-19.

Nothing here is tuned, blocked or fused, and nothing here is shared with the
CUDA path: no common kernels, tables, constants or helpers.  Only the tests,
the smoke check and the benchmark's CPU-baseline leg may import it; the
product must never route through it.

Parity status of each function (what pins it, in tests/test_oracle_*.py):

* basis.gto_alpha, gto_overlap, lowdin, gto_radial ......... pinned
  (threshold identity of Eq. 10, orthonormality by numerical integration,
  brute-force 3-D quadrature of Eq. 3, 40-digit single-neighbour values)
* basis.poly_norm, poly_overlap, poly_radial ............... pinned
  (orthonormality of Eq. 15-17 by quadrature, brute-force 3-D quadrature of
  Eq. 3 over the cutoff sphere, first-order Laplace form Eq. 20 as sigma -> 0)
* harmonics.real_solid_harmonics (+ gradients) ............. pinned
  (SciPy's complex harmonics, Unsold sum rule, Laplace equation, Euler's
  homogeneity relation, finite differences)
* soap.neighbor_list ....................................... pinned
  (brute force over explicit replicas of a periodic cell)
* soap.coefficients / power_spectrum / derivatives ......... pinned
  (Legendre-polynomial closed form free of spherical harmonics, rotation /
  reflection / translation / permutation invariance, central finite
  differences, translation and rotation sum rules of the Jacobian)
* soap.feature_table ....................................... the ORDER of the
  features rests on a reading of the paper's sentence on the nested loops
  (species pair, radial triangle, l fastest); the values do not depend on it.
  With crossover off the table is the mu == nu subset (checked against the
  full table).
* modes.coefficient_vector / coefficient_derivatives ....... pinned
  (the pinned coefficient routine, central finite differences of it, zero
  row sums, zero blocks of foreign species); the ORDER of the coefficient
  index (species, n, l, m) is a reading, the paper names none.
* modes.average_descriptor / average_derivatives ........... pinned
  (bilinear double sum over centre pairs for the inner average, one-centre
  and translation-equivalent-centre reductions to the plain descriptor,
  rotation / permutation invariance, central finite differences)
* modes.site_derivatives (centres that are not atoms) ....... pinned
  (a ghost atom of a species of its own placed at the point, central finite
  differences)
* weighting.weight (radial weighting of the density) ....... pinned
  (brute-force 3-D quadrature of Eq. 3 over weighted Gaussians, central
  finite differences, atoms beyond a vanishing weight drop out, constant
  weight); the functional forms themselves are a reading, the paper names
  the option only.
"""
