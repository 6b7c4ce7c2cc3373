/* soap.h - C ABI of the B200 SOAP descriptor library (libsoap_b200.so).
 *
 * Computes, for every centre atom of a structure, the Smooth Overlap of Atomic
 * Positions partial power spectrum and its analytic Cartesian Jacobian:
 *
 *   neighbours within r_cut (text under Eq. 1)
 *   -> expansion coefficients c^mu_nlm of the Gaussian-smeared species
 *      densities on a radial basis times real spherical harmonics
 *      (Eq. 3; closed form Eq. 13 for Gaussian-type orbitals, the radial
 *      Bessel integral Eqs. 18-19 for polynomials; on-site term included)
 *   -> p^{mu nu}_{n n' l} = pi sqrt(8/(2l+1)) sum_m c^mu_nlm c^nu_n'lm   (Eq. 4)
 *   -> d p / d R_j for every atom j inside the sphere and for the centre
 *      (Eq. 5; Eq. 14 / Eq. 23 for the coefficient gradients).
 *
 * Conventions
 *  - Pointers named d_* are DEVICE pointers owned by the caller; everything
 *    else is host memory.  The handle owns its tables and scratch memory.
 *  - Positions are fp32 Angstrom, row-major [N,3]; atomic numbers int32 [N].
 *  - `cell` is host memory, 9 doubles, rows = lattice vectors a, b, c; it may
 *    be NULL when no axis is periodic.  Positions need not be wrapped.
 *  - `d_centers` lists the centre atoms (indices into the structure); NULL
 *    means every atom, in order (then n_centers must equal n_atoms; n_centers
 *    = 0 is an empty list and does nothing).
 *  - A handle is not thread-safe and serves one stream at a time: its scratch
 *    memory is reused by every call, so calls on one handle must be ordered
 *    (same stream, or synchronised).  Use one handle per concurrent stream or
 *    host thread; handles share nothing but read-only constant tables.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  All
 *    calls enqueue work on it and return without waiting, except where noted.
 *    Within a call the kernels use programmatic dependent launch (each waits on
 *    the device for its predecessor before it reads that kernel's results);
 *    towards other work on the stream a call behaves like any kernel sequence:
 *    its first kernel starts after everything queued before it has finished.
 *  - Feature order: species pairs mu <= nu (species sorted by atomic number),
 *    then the radial pair (n, n') with n' >= n when mu == nu and all n, n'
 *    otherwise (n outer), then l fastest.  F = S n_max (S n_max + 1)/2 (l_max+1).
 *  - Every function returns SOAP_OK or a negative code; nothing throws.
 *    Problems only the device can see (an atomic number outside the species
 *    list, more pairs or rows than a buffer holds) are recorded in a sticky
 *    status word that soap_status() returns after synchronising; when it is
 *    set, the outputs of that call are unspecified.
 *  - The library has no CPU fallback: without a CUDA device the compute
 *    calls return SOAP_ERR_CUDA.
 *  - Arithmetic is fp32 (distances and table offsets fp64, tables built in
 *    quad precision).  Accuracy against an fp64 evaluation of the same
 *    equations, per feature column over the centres of a call: descriptor
 *    within 1e-5 and Jacobian within 1e-4 of the column's largest magnitude,
 *    for every column whose largest magnitude is at least 1e-3 of the largest
 *    entry of the whole output.  A column that is smaller than that for every
 *    centre at once (a few-atom structure whose neighbours all sit near a node
 *    of one radial function, or whose terms cancel) carries the rounding of
 *    the larger quantities it is computed from: its error is bounded relative
 *    to 1e-3 of the output's largest entry, not to its own maximum (in a
 *    500-draw random sweep over structures of 2 to 19 atoms, 489 draws were
 *    within 1e-5 / 1e-4 of that scale and the worst of the others reached
 *    3e-5 / 2e-4; structures of the benchmark sizes meet the column bound
 *    with a margin of 4 to 10).
 */
#ifndef SOAP_B200_H
#define SOAP_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct soap_handle soap_t;

enum {
    SOAP_OK = 0,
    SOAP_ERR_INVALID_ARG = -1,
    SOAP_ERR_UNKNOWN_SPECIES = -2,  /* an atomic number is not in the species list */
    SOAP_ERR_CAPACITY = -3,         /* a caller buffer or the planned scratch is too small */
    SOAP_ERR_CUDA = -4,
    SOAP_ERR_ALLOC = -5
};

enum { SOAP_RBF_GTO = 0, SOAP_RBF_POLYNOMIAL = 1 };

/* Builds a descriptor object: basis constants of Eqs. 8-10 (GTO) or 15-17
 * (polynomial) and the radial tables derived from Eq. 13 / Eqs. 18-19, all on
 * the host in quad precision.  No GPU work happens here; device copies are
 * made on first use.  species: n_species distinct atomic numbers (any order).
 * Limits: 1 <= n_species <= 8, 1 <= n_max <= 16, 0 <= l_max <= 12,
 * r_cut > 0 (> 1 A for GTO, whose width rule Eq. 10 starts at 1 A), sigma > 0.
 * pbc: three flags, one per lattice vector. */
int soap_create(soap_t **out, const int32_t *species, int n_species, double r_cut,
                int n_max, int l_max, double sigma, int rbf, const int pbc[3]);

void soap_destroy(soap_t *h);

/* Number of features F per centre. */
int soap_num_features(const soap_t *h, int64_t *n_features);

/* (mu, nu, n, n', l) of feature f; mu, nu index the sorted species list. */
int soap_feature_info(const soap_t *h, int64_t f, int *mu, int *nu, int *n, int *n2, int *l);

/* Message of the last failing call on this handle (never NULL). */
const char *soap_last_error(const soap_t *h);

/* Host-side check of the radial tables: G_nl(d) and (dG_nl/dd)/d for all
 * n_max*(l_max+1) channels (index n*(l_max+1)+l), where the pair term of
 * Eq. 13 / Eq. 18 is G_nl(d) r^l Y_lm.  Needs no GPU. */
int soap_radial_table(const soap_t *h, double d, double *G, double *Ghat);

/* Neighbour search only (cell list + exact fp64 distance test), then WAITS
 * for the stream.  Returns the number of (centre, neighbour image) pairs and
 * the number of Jacobian rows (distinct atoms per sphere, plus the centre),
 * and sizes the handle's scratch for later calls on structures of this size
 * (with 25% headroom).  Call it before soap_derivatives to size d_jac. */
int soap_neighbors(soap_t *h, const float *d_positions, const int32_t *d_numbers, int64_t n_atoms,
                   const double *cell, const int32_t *d_centers, int64_t n_centers,
                   int64_t *n_pairs, int64_t *n_rows, void *stream);

/* Exports the neighbour list of the last soap_neighbors / soap_descriptor /
 * soap_derivatives call: d_pair_ptr [n_centers+1]; for pair e of centre i
 * (d_pair_ptr[i] <= e < d_pair_ptr[i+1]) the neighbour atom d_pair_atom[e] and
 * its lattice translation d_pair_shift[3e..3e+2] (multiples of a, b, c; may be
 * NULL).  Pairs of a centre are sorted by (atom, shift).  capacity_pairs is
 * the length of the caller's arrays; too small sets SOAP_ERR_CAPACITY. */
int soap_neighbor_list(soap_t *h, int64_t *d_pair_ptr, int32_t *d_pair_atom, int32_t *d_pair_shift,
                       int64_t capacity_pairs, void *stream);

/* Descriptor only: d_out [n_centers, F] fp32, fully overwritten (Eq. 4).
 * Runs the neighbour search itself.  A call for a structure with more atoms
 * or centres than any before it on this handle first plans scratch memory
 * like soap_neighbors (allocates and waits once); other calls only enqueue
 * work.  If such a call meets more pairs than the planned scratch holds (a
 * denser structure), soap_status reports SOAP_ERR_CAPACITY and the outputs
 * of that call are invalid: call soap_neighbors for that structure, then
 * repeat. */
int soap_descriptor(soap_t *h, const float *d_positions, const int32_t *d_numbers, int64_t n_atoms,
                    const double *cell, const int32_t *d_centers, int64_t n_centers,
                    float *d_out, void *stream);

/* Descriptor and Jacobian (Eqs. 4 and 5).  Runs the neighbour search itself.
 *   d_out_desc [n_centers, F]
 *   d_row_ptr  [n_centers+1]   rows of centre i are d_row_ptr[i] .. d_row_ptr[i+1]-1
 *   d_row_atom [capacity_rows] atom each row differentiates with respect to;
 *                              ascending within a centre, the centre included
 *   d_out_jac  [capacity_rows, 3, F]  d p_f / d (x,y,z of that atom); all other
 *              entries of the dense (centre, atom, 3, F) Jacobian are zero.
 * Periodic images of one atom add up in that atom's row.  Every row below
 * d_row_ptr[n_centers] is fully overwritten.  If the structure has more rows
 * than capacity_rows nothing is written and the status becomes
 * SOAP_ERR_CAPACITY. */
int soap_derivatives(soap_t *h, const float *d_positions, const int32_t *d_numbers, int64_t n_atoms,
                     const double *cell, const int32_t *d_centers, int64_t n_centers,
                     float *d_out_desc, float *d_out_jac, int64_t capacity_rows,
                     int64_t *d_row_ptr, int32_t *d_row_atom, void *stream);

/* Dense view of the Jacobian in the layout of the paper's derivatives() call
 * (architecture section: (n_centers, n_atoms, 3, n_features)), for the atoms of
 * an inclusion list:
 *   d_out [n_centers, n_include, 3, F]   fully overwritten; the block of
 *         (centre c, listed atom a) is that atom's row of centre c, or zeros
 *         when the atom is outside the centre's sphere (the text below Eq. 5:
 *         only atoms inside the cutoff contribute).
 *   d_include [n_include] atom indices, or NULL for atoms 0 .. n_include-1
 *         (pass n_include = n_atoms for the paper's full layout; leaving atoms
 *         out of the list is its `exclude`).
 * d_jac_rows / d_row_ptr / d_row_atom are the outputs of soap_derivatives for
 * the same n_centers.  The dense tensor grows as centres x atoms: meant for
 * small structures or for batches of centres.  n_centers * n_include must stay
 * below 2^31. */
int soap_jacobian_dense(soap_t *h, const float *d_jac_rows, const int64_t *d_row_ptr, const int32_t *d_row_atom,
                        int64_t n_centers, const int32_t *d_include, int64_t n_include, float *d_out, void *stream);

/* The same scatter for rows of any width (`width` floats per direction): the
 * dense (centre, atom, 3, W) view of soap_coefficient_derivatives' rows. */
int soap_rows_dense(soap_t *h, const float *d_rows, int64_t width, const int64_t *d_row_ptr, const int32_t *d_row_atom,
                    int64_t n_centers, const int32_t *d_include, int64_t n_include, float *d_out, void *stream);

/* ---- output modes beyond the per-centre power spectrum (the interface section of the
 *      paper: the crossover flag, the coefficient mode, the inner and outer averages) ---- */

/* crossover = 0 keeps only the species pairs mu == nu (F = S n(n+1)/2 (l+1));
 * the default keeps every pair mu <= nu.  Changes soap_num_features and
 * soap_feature_info; waits for the device when tables are already uploaded.
 * Not to be called while work on this handle is in flight. */
int soap_set_crossover(soap_t *h, int crossover);

/* ---- many independent structures in one call ----
 * The paper enumerates work as batches of centres drawn from one structure
 * each and notes that small systems are bound by launch latency.  These entry
 * points take many non-periodic structures as ONE list of atoms:
 * d_struct_ptr [n_structs+1] (device, ascending, d_struct_ptr[0] = 0,
 * d_struct_ptr[n_structs] = n_atoms) delimits the structures; every atom is a
 * centre and sees only the atoms of its own structure (0 < d^2 < r_cut^2,
 * the same fp64 test), found by a warp running over that structure - meant for
 * molecules of up to a few hundred atoms.  Outputs as in soap_descriptor /
 * soap_derivatives with atom and centre indices counted through the whole
 * list; the launch count does not depend on the number of structures.  The
 * handle must have no periodic axis.  Planning, capacities and errors as in
 * soap_neighbors / soap_derivatives. */
int soap_neighbors_batch(soap_t *h, const float *d_positions, const int32_t *d_numbers, int64_t n_atoms,
                         const int64_t *d_struct_ptr, int64_t n_structs, int64_t *n_pairs, int64_t *n_rows,
                         void *stream);
int soap_descriptor_batch(soap_t *h, const float *d_positions, const int32_t *d_numbers, int64_t n_atoms,
                          const int64_t *d_struct_ptr, int64_t n_structs, float *d_out, void *stream);
int soap_derivatives_batch(soap_t *h, const float *d_positions, const int32_t *d_numbers, int64_t n_atoms,
                           const int64_t *d_struct_ptr, int64_t n_structs, float *d_out_desc, float *d_out_jac,
                           int64_t capacity_rows, int64_t *d_row_ptr, int32_t *d_row_atom, void *stream);

/* ---- species-compact Jacobian rows ----
 * The row of a neighbour of species Z is zero in every species-pair block that
 * does not involve Z (Eq. 5: grad_j c^mu vanishes unless atom j has species mu;
 * the paper's kernels write those zeros explicitly).  The compact format leaves
 * them out: a neighbour row holds, in feature order, only the blocks (mu, nu)
 * with mu == Z or nu == Z: n_compact = one same-species block + (S-1) cross
 * blocks, the same for every Z, against F = S same-species + S(S-1)/2 cross
 * blocks.  Rows are stored with a pitch of n_compact rounded up to a multiple
 * of 8 floats (padding written as zeros).  The centre's own row involves every
 * block and goes, full width, to an array of its own. */
int soap_num_compact_features(const soap_t *h, int64_t *n_compact, int64_t *pitch);

/* map[j] = index of the full feature that column j of a compact row of species
 * `species_index` (position in the sorted species list) holds; host memory,
 * n_compact entries, ascending. */
int soap_compact_feature_map(const soap_t *h, int species_index, int32_t *map);

/* soap_derivatives with compact rows:
 *   d_out_center [n_centers, 3, F]         the centre's own row (all blocks)
 *   d_out_jac    [capacity_rows, 3, pitch] neighbour rows, compact; the slot of
 *                the centre's own row (row_atom == the centre) is zero-filled
 * row_ptr / row_atom / d_out_desc / errors as in soap_derivatives. */
int soap_derivatives_compact(soap_t *h, const float *d_positions, const int32_t *d_numbers, int64_t n_atoms,
                             const double *cell, const int32_t *d_centers, int64_t n_centers,
                             float *d_out_desc, float *d_out_center, float *d_out_jac, int64_t capacity_rows,
                             int64_t *d_row_ptr, int32_t *d_row_atom, void *stream);

/* Expands compact rows to the full rows soap_derivatives writes:
 * d_out_rows [n_rows, 3, F].  d_centers as in the producing call (NULL = all
 * atoms); d_numbers the structure's atomic numbers. */
int soap_compact_expand(soap_t *h, const int32_t *d_numbers, const int32_t *d_centers, int64_t n_centers,
                        const float *d_center_rows, const float *d_jac_compact, const int64_t *d_row_ptr,
                        const int32_t *d_row_atom, float *d_out_rows, void *stream);

/* Centres at arbitrary points instead of at atoms (the interface accepts an
 * explicit list of centres): d_sites [n_sites, 3] fp32 Cartesian, device.  A
 * point has no Gaussian of its own, so there is no on-site term (Eq. 13, second
 * term) and no Jacobian row for the centre: rows are the atoms in the sphere
 * only.  A point that coincides with an atom drops that atom (the neighbour
 * test is 0 < d^2): pass the atom as a centre to soap_derivatives instead.
 * Everything else (arguments, sizing with soap_neighbors_at, errors, status)
 * as in soap_neighbors / soap_descriptor / soap_derivatives. */
int soap_neighbors_at(soap_t *h, const float *d_positions, const int32_t *d_numbers, int64_t n_atoms,
                      const double *cell, const float *d_sites, int64_t n_sites,
                      int64_t *n_pairs, int64_t *n_rows, void *stream);
int soap_descriptor_at(soap_t *h, const float *d_positions, const int32_t *d_numbers, int64_t n_atoms,
                       const double *cell, const float *d_sites, int64_t n_sites, float *d_out, void *stream);
int soap_derivatives_at(soap_t *h, const float *d_positions, const int32_t *d_numbers, int64_t n_atoms,
                        const double *cell, const float *d_sites, int64_t n_sites,
                        float *d_out_desc, float *d_out_jac, int64_t capacity_rows,
                        int64_t *d_row_ptr, int32_t *d_row_atom, void *stream);

enum { SOAP_WEIGHT_NONE = 0, SOAP_WEIGHT_POLY = 1, SOAP_WEIGHT_POW = 2, SOAP_WEIGHT_EXP = 3 };

/* Radial weighting of the neighbour density (the `weighting` argument of the
 * paper's constructor, which names the option and gives no formula; the forms
 * are our reading): the Gaussian of a neighbour at distance dist from the
 * centre (Eq. 1) is scaled by
 *   POLY: c (1 + 2 x^3 - 3 x^2)^m for x = dist/r0 <= 1, else 0   (d unused)
 *   POW:  c / (d + x^m)
 *   EXP:  c / (d + exp(-x))                                         (m unused)
 * and the centre's own Gaussian (on-site term of Eq. 13) by w0.  The weight
 * multiplies the neighbour's whole term, so the Jacobian gains the product-rule
 * term w'(dist).  Evaluated per pair in fp64 by a kernel of its own after the
 * neighbour search.  SOAP_WEIGHT_NONE switches it off.  Not to be called while
 * work on this handle is in flight (it may wait for the device and reallocate). */
int soap_set_weighting(soap_t *h, int function, double r0, double c, double d, double m, double w0);

/* Number of expansion coefficients per centre, W = S n_max (l_max+1)^2. */
int soap_num_coefficients(const soap_t *h, int64_t *n_coefficients);

/* Coefficient mode: the projection coefficients c^mu_nlm of Eq. 3 themselves
 * (Eq. 13 / Eq. 18, on-site term included) instead of their contraction.
 * d_out [n_centers, W], index (mu n_max + n)(l_max+1)^2 + l^2 + l + m with the
 * real spherical harmonics m = -l..l (the paper fixes no order: this one is
 * ours).  Otherwise like soap_descriptor. */
int soap_coefficients(soap_t *h, const float *d_positions, const int32_t *d_numbers, int64_t n_atoms,
                      const double *cell, const int32_t *d_centers, int64_t n_centers,
                      float *d_out, void *stream);

/* Coefficients and their Jacobian d c^mu_nlm / d R_j (Eq. 14 / Eq. 23) in the
 * row format of soap_derivatives with W in place of F: d_out_coeff
 * [n_centers, W], d_out_jac [capacity_rows, 3, W].  A neighbour's row is
 * non-zero only in the block of its own species; the centre's row is minus
 * the sum of the others.  Errors and capacities as in soap_derivatives. */
int soap_coefficient_derivatives(soap_t *h, const float *d_positions, const int32_t *d_numbers, int64_t n_atoms,
                                 const double *cell, const int32_t *d_centers, int64_t n_centers,
                                 float *d_out_coeff, float *d_out_jac, int64_t capacity_rows,
                                 int64_t *d_row_ptr, int32_t *d_row_atom, void *stream);

enum { SOAP_AVERAGE_INNER = 1, SOAP_AVERAGE_OUTER = 2 };

/* One averaged descriptor for the whole centre list, d_out [F]:
 *   outer: the mean over the centres of their power spectra (Eq. 4);
 *   inner: Eq. 4 applied to the mean over the centres of c^mu_nlm.
 * n_centers >= 1.  Sums run in a fixed order (results repeat bit for bit).
 * The handle keeps a workspace of n_centers max(F, W) floats. */
int soap_descriptor_average(soap_t *h, int mode, const float *d_positions, const int32_t *d_numbers,
                            int64_t n_atoms, const double *cell, const int32_t *d_centers,
                            int64_t n_centers, float *d_out, void *stream);

/* Averaged descriptor d_out_desc [F] and its Jacobian with respect to EVERY
 * atom, d_out_jac [n_atoms, 3, F], fully overwritten (zero rows for atoms in
 * no centre's sphere).  The per-centre rows (Eq. 5; for the inner average
 * taken against the mean coefficients) go to a workspace inside the handle of
 * n_rows 3 F floats, n_rows as soap_neighbors reports it, and are then summed
 * per atom in centre order; SOAP_ERR_ALLOC when that does not fit the device
 * (split the centre list and average the partial results by their weights).
 * WAITS for the stream once (it reads the row total). */
int soap_derivatives_average(soap_t *h, int mode, const float *d_positions, const int32_t *d_numbers,
                             int64_t n_atoms, const double *cell, const int32_t *d_centers,
                             int64_t n_centers, float *d_out_desc, float *d_out_jac, void *stream);

/* Waits for `stream`, then returns and clears the sticky device status
 * (SOAP_OK, SOAP_ERR_UNKNOWN_SPECIES or SOAP_ERR_CAPACITY); also reports the
 * pair and row counts of the last call (either pointer may be NULL).  The
 * descriptor-only calls build no Jacobian rows and keep their pairs unsorted:
 * after one of them the row count is zero and soap_neighbor_list wants a
 * soap_neighbors call first. */
int soap_status(soap_t *h, int64_t *n_pairs, int64_t *n_rows, void *stream);

/* Measurement aid (the paper has no counterpart): the FP32 multiply-add rate of
 * the current device from a register-only loop (16 independent chains per
 * thread, 8 CTAs of 256 threads per SM, about 20 ms), timed with CUDA events on
 * `stream`; the call waits for it.  *tflops receives 2 x multiply-adds / time
 * of the best of four repetitions, *milliseconds (may be NULL) that time.
 * This is the denominator the descriptor-only build is measured against. */
int soap_measure_fp32_peak(double *tflops, double *milliseconds, void *stream);

/* Neighbour counts with NO allocation anywhere in the call (the paper has no
 * counterpart; this entry point exists for callers that must not allocate).
 * Some callers cannot call cudaMalloc, or anything that may: a host
 * application that gave its whole device-memory budget to its own pool at
 * start-up, a latency-critical loop that cannot afford the implicit device
 * synchronisation of an allocation, or a plug-in that is forbidden to touch
 * the allocator of the process it lives in.  For them this call counts, for
 * every atom of a NON-PERIODIC structure, the atoms within r_cut
 * (0 < distance^2 < r_cut^2, the same exact fp64 test and the same cell-list
 * kernels as soap_neighbors), keeping the cell list in a fixed array compiled
 * into the library instead of allocated scratch.
 *   d_positions [n_atoms,3] fp32, device   (input, caller-owned)
 *   d_counts    [n_atoms]   int32, device  (output, caller-owned, fully overwritten)
 *   message     optional host buffer of message_len bytes for the error text
 * Limit: n_atoms <= 65536; more returns SOAP_ERR_CAPACITY and does nothing.
 * Cost of the limit: about 2.4 MB of device memory on every GPU that loads the
 * library, held until the process exits.
 * The call uses no handle, calls no cudaMalloc / cudaFree / allocating library
 * routine, and enqueues its work on `stream` without waiting.  The first call
 * on a device also looks up the device address of the fixed array (once per
 * device, with that device current); make that first call outside any stream
 * capture.  The looked-up address is cached per device and published
 * atomically, so host threads may race on their first calls; it goes stale if
 * the device is reset (cudaDeviceReset) while the library stays loaded.  All calls on one GPU share the one array, which keeps the last
 * call's contents (the call clears what must start at zero): two calls whose
 * work overlaps on the GPU - different streams, or different host threads on
 * different streams - race on it and give wrong counts.  Serialise them. */
int soap_neighbor_counts_static(const float *d_positions, int64_t n_atoms, double r_cut,
                                int32_t *d_counts, void *stream, char *message, int64_t message_len);

/* Per-segment timing, the counterpart of the paper's companion profiler
 * (end of its architecture section).  With profiling enabled,
 * soap_descriptor and soap_derivatives record CUDA events on the caller's
 * stream around (a) the neighbour search and (b) the fused per-centre kernel.
 * soap_profile_read waits for the last call's events and returns both
 * durations in milliseconds.  Off by default: the kernels of a call are
 * launched so that each may start while the one before it finishes (they wait
 * for it on the device), and an event recorded between two launches keeps the
 * second from starting early - a profiled call is a few microseconds slower,
 * and its two durations can add up to more than an unprofiled call takes. */
int soap_profile(soap_t *h, int enable);
int soap_profile_read(soap_t *h, float *ms_neighbors, float *ms_center);

#ifdef __cplusplus
}
#endif
#endif /* SOAP_B200_H */
