"""ctypes binding of libsoap_b200.so (argument marshalling only)."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np

GTO, POLYNOMIAL = 0, 1
AVERAGE_MODES = {"inner": 1, "outer": 2}
WEIGHT_FUNCTIONS = {"poly": 1, "pow": 2, "exp": 3}

EXPORTED_SYMBOLS = [
    "soap_create", "soap_destroy", "soap_num_features", "soap_feature_info", "soap_last_error",
    "soap_radial_table", "soap_neighbors", "soap_neighbor_list", "soap_descriptor",
    "soap_derivatives", "soap_status", "soap_profile", "soap_profile_read", "soap_neighbor_counts_static", "soap_jacobian_dense",
    "soap_set_crossover", "soap_num_coefficients", "soap_coefficients", "soap_coefficient_derivatives",
    "soap_descriptor_average", "soap_derivatives_average", "soap_set_weighting",
    "soap_neighbors_at", "soap_descriptor_at", "soap_derivatives_at",
    "soap_rows_dense", "soap_neighbors_batch", "soap_descriptor_batch", "soap_derivatives_batch",
    "soap_num_compact_features", "soap_compact_feature_map", "soap_derivatives_compact", "soap_compact_expand",
    "soap_measure_fp32_peak",
]

_ERRORS = {-1: "SOAP_ERR_INVALID_ARG", -2: "SOAP_ERR_UNKNOWN_SPECIES", -3: "SOAP_ERR_CAPACITY",
           -4: "SOAP_ERR_CUDA", -5: "SOAP_ERR_ALLOC"}


class SoapError(RuntimeError):
    def __init__(self, code, message):
        super().__init__(f"{_ERRORS.get(code, code)}: {message}")
        self.code = code


def library_path() -> str:
    """The in-tree build, unless SOAP_B200_LIB names another build of the same library."""
    return os.environ.get("SOAP_B200_LIB") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libsoap_b200.so")


_LIB = None


def load_library() -> C.CDLL:
    """Loads the shared library (never builds it, never falls back)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2609_05709_b200.build`")
    lib = C.CDLL(path)
    vp, i64, i32 = C.c_void_p, C.c_int64, C.c_int
    lib.soap_create.argtypes = [C.POINTER(vp), C.POINTER(C.c_int32), i32, C.c_double, i32, i32, C.c_double, i32, C.POINTER(i32)]
    lib.soap_destroy.argtypes = [vp]
    lib.soap_destroy.restype = None
    lib.soap_num_features.argtypes = [vp, C.POINTER(i64)]
    lib.soap_feature_info.argtypes = [vp, i64] + [C.POINTER(i32)] * 5
    lib.soap_last_error.argtypes = [vp]
    lib.soap_last_error.restype = C.c_char_p
    lib.soap_radial_table.argtypes = [vp, C.c_double, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    common = [vp, vp, vp, i64, C.POINTER(C.c_double), vp, i64]
    lib.soap_neighbors.argtypes = common + [C.POINTER(i64), C.POINTER(i64), vp]
    lib.soap_neighbor_list.argtypes = [vp, vp, vp, vp, i64, vp]
    lib.soap_descriptor.argtypes = common + [vp, vp]
    lib.soap_derivatives.argtypes = common + [vp, vp, i64, vp, vp, vp]
    lib.soap_status.argtypes = [vp, C.POINTER(i64), C.POINTER(i64), vp]
    lib.soap_neighbor_counts_static.argtypes = [vp, i64, C.c_double, vp, vp, C.c_char_p, i64]
    lib.soap_jacobian_dense.argtypes = [vp, vp, vp, vp, i64, vp, i64, vp, vp]
    lib.soap_rows_dense.argtypes = [vp, vp, i64, vp, vp, i64, vp, i64, vp, vp]
    lib.soap_neighbors_at.argtypes = common + [C.POINTER(i64), C.POINTER(i64), vp]
    lib.soap_descriptor_at.argtypes = common + [vp, vp]
    lib.soap_derivatives_at.argtypes = common + [vp, vp, i64, vp, vp, vp]
    lib.soap_num_compact_features.argtypes = [vp, C.POINTER(i64), C.POINTER(i64)]
    lib.soap_compact_feature_map.argtypes = [vp, i32, C.POINTER(C.c_int32)]
    lib.soap_derivatives_compact.argtypes = common + [vp, vp, vp, i64, vp, vp, vp]
    lib.soap_compact_expand.argtypes = [vp, vp, vp, i64, vp, vp, vp, vp, vp, vp]
    lib.soap_neighbors_batch.argtypes = [vp, vp, vp, i64, vp, i64, C.POINTER(i64), C.POINTER(i64), vp]
    lib.soap_descriptor_batch.argtypes = [vp, vp, vp, i64, vp, i64, vp, vp]
    lib.soap_derivatives_batch.argtypes = [vp, vp, vp, i64, vp, i64, vp, vp, i64, vp, vp, vp]
    lib.soap_set_crossover.argtypes = [vp, i32]
    lib.soap_set_weighting.argtypes = [vp, i32] + [C.c_double] * 5
    lib.soap_num_coefficients.argtypes = [vp, C.POINTER(i64)]
    lib.soap_coefficients.argtypes = common + [vp, vp]
    lib.soap_coefficient_derivatives.argtypes = common + [vp, vp, i64, vp, vp, vp]
    lib.soap_descriptor_average.argtypes = [vp, i32] + common[1:] + [vp, vp]
    lib.soap_derivatives_average.argtypes = [vp, i32] + common[1:] + [vp, vp, vp]
    lib.soap_measure_fp32_peak.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_double), vp]
    lib.soap_profile.argtypes = [vp, i32]
    lib.soap_profile_read.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_float)]
    for name in EXPORTED_SYMBOLS:
        if name not in ("soap_destroy", "soap_last_error"):
            getattr(lib, name).restype = C.c_int
    _LIB = lib
    return lib


def measure_fp32_peak():
    """(TFLOP/s, ms) of the library's register-only FP32 multiply-add loop on the current device and stream."""
    import torch
    lib = load_library()
    tf, ms = C.c_double(), C.c_double()
    rc = lib.soap_measure_fp32_peak(C.byref(tf), C.byref(ms), C.c_void_p(torch.cuda.current_stream().cuda_stream))
    if rc != 0:
        raise SoapError(rc, "soap_measure_fp32_peak failed (is a CUDA device present?)")
    return tf.value, ms.value


def neighbor_counts_static(positions, r_cut, out=None):
    """Atoms within r_cut of every atom of a non-periodic structure, through the entry point that
    allocates nothing inside the library (at most 65536 atoms; the output tensor is the caller's:
    pass `out` to keep this wrapper allocation-free as well).  Work is enqueued on the current
    stream; calls that overlap on the GPU race on the library's fixed scratch array."""
    import torch
    lib = load_library()
    assert positions.is_cuda and positions.dtype == torch.float32 and positions.is_contiguous()
    n = positions.shape[0]
    if out is None:
        out = torch.empty(n, dtype=torch.int32, device=positions.device)
    msg = C.create_string_buffer(256)
    rc = lib.soap_neighbor_counts_static(positions.data_ptr(), n, float(r_cut), out.data_ptr(),
                                         C.c_void_p(torch.cuda.current_stream().cuda_stream), msg, 256)
    if rc != 0:
        raise SoapError(rc, msg.value.decode())
    return out


@dataclass
class CompactDerivatives:
    descriptor: "torch.Tensor"   # (C, F)
    center_rows: "torch.Tensor"  # (C, 3, F) the centre's own row
    jacobian: "torch.Tensor"     # (rows, 3, pitch) species-compact neighbour rows
    row_ptr: "torch.Tensor"      # (C+1,)
    row_atom: "torch.Tensor"     # (rows,)


@dataclass
class Derivatives:
    descriptor: "torch.Tensor"   # (C, F) float32, device
    jacobian: "torch.Tensor"     # (rows, 3, F) float32, device
    row_ptr: "torch.Tensor"      # (C+1,) int64, device
    row_atom: "torch.Tensor"     # (rows,) int32, device


class Soap:
    """One descriptor configuration (the arguments of soap_create)."""

    def __init__(self, species, r_cut, n_max, l_max, sigma, rbf=GTO, pbc=(False, False, False), crossover=True,
                 weighting=None):
        """`weighting`: None or {"function": "poly" | "pow" | "exp", "r0", "c", "m", "d", "w0"} (see
        soap_set_weighting in include/soap.h)."""
        self._lib = load_library()
        self._h = C.c_void_p()
        sp = (C.c_int32 * len(species))(*[int(z) for z in species])
        pb = (C.c_int * 3)(*[int(bool(p)) for p in pbc])
        rc = self._lib.soap_create(C.byref(self._h), sp, len(species), float(r_cut), int(n_max), int(l_max),
                                   float(sigma), int(rbf), pb)
        if rc != 0:
            msg = self._lib.soap_last_error(self._h).decode() if self._h else "allocation failed"
            self.close()
            raise SoapError(rc, msg)
        n = C.c_int64()
        if not crossover:
            self._check(self._lib.soap_set_crossover(self._h, 0))
        if weighting:
            self._check(self._lib.soap_set_weighting(
                self._h, WEIGHT_FUNCTIONS[weighting["function"]], float(weighting["r0"]), float(weighting.get("c", 1.0)),
                float(weighting.get("d", 1.0)), float(weighting.get("m", 1.0)), float(weighting.get("w0", 1.0))))
        self._check(self._lib.soap_num_features(self._h, C.byref(n)))
        self.n_features = int(n.value)
        self._check(self._lib.soap_num_coefficients(self._h, C.byref(n)))
        self.n_coefficients = int(n.value)
        pitch = C.c_int64()
        self._check(self._lib.soap_num_compact_features(self._h, C.byref(n), C.byref(pitch)))
        self.n_compact, self.compact_pitch = int(n.value), int(pitch.value)
        self.n_channels = int(n_max) * (int(l_max) + 1)
        self.pbc = tuple(bool(p) for p in pbc)

    # ------------------------------------------------------------------ plumbing
    def close(self):
        if getattr(self, "_h", None):
            self._lib.soap_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc):
        if rc != 0:
            raise SoapError(rc, self._lib.soap_last_error(self._h).decode())

    @staticmethod
    def _stream():
        import torch
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)

    @staticmethod
    def _cell(cell):
        if cell is None:
            return None, None
        arr = np.ascontiguousarray(np.asarray(cell, np.float64).reshape(9))
        return arr, arr.ctypes.data_as(C.POINTER(C.c_double))

    @staticmethod
    def _inputs(positions, numbers, centers):
        import torch
        assert positions.is_cuda and positions.dtype == torch.float32 and positions.is_contiguous()
        assert numbers.is_cuda and numbers.dtype == torch.int32 and numbers.is_contiguous()
        n = positions.shape[0]
        if centers is None:
            return n, n, None
        assert centers.is_cuda and centers.dtype == torch.int32 and centers.is_contiguous()
        return n, centers.shape[0], C.c_void_p(centers.data_ptr())

    # ------------------------------------------------------------------ host-only helpers
    def feature_info(self, f):
        out = [C.c_int() for _ in range(5)]
        self._check(self._lib.soap_feature_info(self._h, int(f), *[C.byref(o) for o in out]))
        return tuple(o.value for o in out)      # mu, nu, n, n', l

    def radial_table(self, d):
        G = np.empty(self.n_channels)
        Gh = np.empty(self.n_channels)
        self._check(self._lib.soap_radial_table(self._h, float(d), G.ctypes.data_as(C.POINTER(C.c_double)),
                                                Gh.ctypes.data_as(C.POINTER(C.c_double))))
        return G, Gh

    # ------------------------------------------------------------------ device calls
    def neighbors(self, positions, numbers, cell=None, centers=None):
        """(n_pairs, n_rows); waits for the stream."""
        n, c, cptr = self._inputs(positions, numbers, centers)
        keep, cellp = self._cell(cell)
        npairs, nrows = C.c_int64(), C.c_int64()
        self._check(self._lib.soap_neighbors(self._h, positions.data_ptr(), numbers.data_ptr(), n, cellp, cptr, c,
                                             C.byref(npairs), C.byref(nrows), self._stream()))
        return int(npairs.value), int(nrows.value)

    def neighbor_list(self, positions, numbers, cell=None, centers=None):
        """pair_ptr (C+1,), pair_atom (E,), pair_shift (E,3) as device tensors."""
        import torch
        npairs, _ = self.neighbors(positions, numbers, cell, centers)
        c = positions.shape[0] if centers is None else centers.shape[0]
        ptr = torch.empty(c + 1, dtype=torch.int64, device=positions.device)
        atom = torch.empty(max(npairs, 1), dtype=torch.int32, device=positions.device)
        shift = torch.empty((max(npairs, 1), 3), dtype=torch.int32, device=positions.device)
        self._check(self._lib.soap_neighbor_list(self._h, ptr.data_ptr(), atom.data_ptr(), shift.data_ptr(), npairs, self._stream()))
        self.status()
        return ptr, atom[:npairs], shift[:npairs]

    def descriptor(self, positions, numbers, cell=None, centers=None, out=None):
        import torch
        n, c, cptr = self._inputs(positions, numbers, centers)
        keep, cellp = self._cell(cell)
        if out is None:
            out = torch.empty((c, self.n_features), dtype=torch.float32, device=positions.device)
        self._check(self._lib.soap_descriptor(self._h, positions.data_ptr(), numbers.data_ptr(), n, cellp, cptr, c,
                                              out.data_ptr(), self._stream()))
        return out

    def derivatives_into(self, positions, numbers, cell, centers, desc, jac, row_ptr, row_atom):
        """Asynchronous call into caller-provided buffers (jac: (capacity_rows, 3, F))."""
        n, c, cptr = self._inputs(positions, numbers, centers)
        keep, cellp = self._cell(cell)
        self._check(self._lib.soap_derivatives(self._h, positions.data_ptr(), numbers.data_ptr(), n, cellp, cptr, c,
                                               desc.data_ptr(), jac.data_ptr(), jac.shape[0], row_ptr.data_ptr(),
                                               row_atom.data_ptr(), self._stream()))

    def derivatives(self, positions, numbers, cell=None, centers=None) -> Derivatives:
        """Sizes the Jacobian with one neighbour search, then computes it."""
        import torch
        _, nrows = self.neighbors(positions, numbers, cell, centers)
        c = positions.shape[0] if centers is None else centers.shape[0]
        dev = positions.device
        desc = torch.empty((c, self.n_features), dtype=torch.float32, device=dev)
        jac = torch.empty((max(nrows, 1), 3, self.n_features), dtype=torch.float32, device=dev)
        row_ptr = torch.empty(c + 1, dtype=torch.int64, device=dev)
        row_atom = torch.empty(max(nrows, 1), dtype=torch.int32, device=dev)
        self.derivatives_into(positions, numbers, cell, centers, desc, jac, row_ptr, row_atom)
        self.status()
        return Derivatives(desc, jac[:nrows], row_ptr, row_atom[:nrows])

    # ------------------------------------------------------------------ many structures in one call
    def derivatives_batch(self, positions, numbers, struct_ptr, jacobian=True):
        """Many independent non-periodic structures as one list of atoms; `struct_ptr` is an int64 device
        tensor (B+1,) of offsets.  Returns `Derivatives` over all atoms (indices through the whole list), or
        the (N, F) descriptor with jacobian=False."""
        import torch
        n, _, _ = self._inputs(positions, numbers, None)
        assert struct_ptr.is_cuda and struct_ptr.dtype == torch.int64 and struct_ptr.is_contiguous()
        b, sp = struct_ptr.shape[0] - 1, C.c_void_p(struct_ptr.data_ptr())
        dev = positions.device
        desc = torch.empty((n, self.n_features), dtype=torch.float32, device=dev)
        if not jacobian:
            self._check(self._lib.soap_descriptor_batch(self._h, positions.data_ptr(), numbers.data_ptr(), n, sp, b,
                                                        desc.data_ptr(), self._stream()))
            self.status()
            return desc
        npairs, nrows = C.c_int64(), C.c_int64()
        self._check(self._lib.soap_neighbors_batch(self._h, positions.data_ptr(), numbers.data_ptr(), n, sp, b,
                                                   C.byref(npairs), C.byref(nrows), self._stream()))
        nrows = int(nrows.value)
        jac = torch.empty((max(nrows, 1), 3, self.n_features), dtype=torch.float32, device=dev)
        row_ptr = torch.empty(n + 1, dtype=torch.int64, device=dev)
        row_atom = torch.empty(max(nrows, 1), dtype=torch.int32, device=dev)
        self._check(self._lib.soap_derivatives_batch(self._h, positions.data_ptr(), numbers.data_ptr(), n, sp, b,
                                                     desc.data_ptr(), jac.data_ptr(), jac.shape[0], row_ptr.data_ptr(),
                                                     row_atom.data_ptr(), self._stream()))
        self.status()
        return Derivatives(desc, jac[:nrows], row_ptr, row_atom[:nrows])

    # ------------------------------------------------------------------ species-compact rows
    def compact_feature_map(self, species_index):
        out = np.empty(self.n_compact, np.int32)
        self._check(self._lib.soap_compact_feature_map(self._h, int(species_index), out.ctypes.data_as(C.POINTER(C.c_int32))))
        return out

    def derivatives_compact_into(self, positions, numbers, cell, centers, desc, center_rows, jac, row_ptr, row_atom):
        n, c, cptr = self._inputs(positions, numbers, centers)
        keep, cellp = self._cell(cell)
        self._check(self._lib.soap_derivatives_compact(self._h, positions.data_ptr(), numbers.data_ptr(), n, cellp, cptr, c,
                                                       desc.data_ptr(), center_rows.data_ptr(), jac.data_ptr(), jac.shape[0],
                                                       row_ptr.data_ptr(), row_atom.data_ptr(), self._stream()))

    def derivatives_compact(self, positions, numbers, cell=None, centers=None) -> CompactDerivatives:
        """Like `derivatives`, with neighbour rows that leave out the structurally zero species blocks."""
        import torch
        _, nrows = self.neighbors(positions, numbers, cell, centers)
        c = positions.shape[0] if centers is None else centers.shape[0]
        dev = positions.device
        desc = torch.empty((c, self.n_features), dtype=torch.float32, device=dev)
        center_rows = torch.empty((c, 3, self.n_features), dtype=torch.float32, device=dev)
        jac = torch.empty((max(nrows, 1), 3, self.compact_pitch), dtype=torch.float32, device=dev)
        row_ptr = torch.empty(c + 1, dtype=torch.int64, device=dev)
        row_atom = torch.empty(max(nrows, 1), dtype=torch.int32, device=dev)
        self.derivatives_compact_into(positions, numbers, cell, centers, desc, center_rows, jac, row_ptr, row_atom)
        self.status()
        return CompactDerivatives(desc, center_rows, jac[:nrows], row_ptr, row_atom[:nrows])

    def compact_expand(self, numbers, centers, comp: "CompactDerivatives"):
        """(rows, 3, F): the full rows `derivatives` would have written."""
        import torch
        rows = comp.jacobian.shape[0]
        out = torch.empty((max(rows, 1), 3, self.n_features), dtype=torch.float32, device=comp.jacobian.device)
        c = comp.row_ptr.shape[0] - 1
        cptr = None if centers is None else C.c_void_p(centers.data_ptr())
        self._check(self._lib.soap_compact_expand(self._h, numbers.data_ptr(), cptr, c, comp.center_rows.data_ptr(),
                                                  comp.jacobian.data_ptr(), comp.row_ptr.data_ptr(), comp.row_atom.data_ptr(),
                                                  out.data_ptr(), self._stream()))
        return out[:rows]

    # ------------------------------------------------------------------ centres that are not atoms
    def derivatives_at(self, positions, numbers, sites, cell=None, jacobian=True):
        """Descriptor (and Jacobian) for centres at the points `sites` (float32 device tensor (C, 3)):
        no on-site term and no row for the centre itself.  Returns `Derivatives`, or the (C, F)
        descriptor with jacobian=False."""
        import torch
        n, _, _ = self._inputs(positions, numbers, None)
        assert sites.is_cuda and sites.dtype == torch.float32 and sites.is_contiguous() and sites.shape[-1] == 3
        c, sptr = sites.shape[0], C.c_void_p(sites.data_ptr())
        keep, cellp = self._cell(cell)
        dev = positions.device
        desc = torch.empty((c, self.n_features), dtype=torch.float32, device=dev)
        if not jacobian:
            self._check(self._lib.soap_descriptor_at(self._h, positions.data_ptr(), numbers.data_ptr(), n, cellp, sptr, c,
                                                     desc.data_ptr(), self._stream()))
            self.status()
            return desc
        npairs, nrows = C.c_int64(), C.c_int64()
        self._check(self._lib.soap_neighbors_at(self._h, positions.data_ptr(), numbers.data_ptr(), n, cellp, sptr, c,
                                                C.byref(npairs), C.byref(nrows), self._stream()))
        nrows = int(nrows.value)
        jac = torch.empty((max(nrows, 1), 3, self.n_features), dtype=torch.float32, device=dev)
        row_ptr = torch.empty(c + 1, dtype=torch.int64, device=dev)
        row_atom = torch.empty(max(nrows, 1), dtype=torch.int32, device=dev)
        self._check(self._lib.soap_derivatives_at(self._h, positions.data_ptr(), numbers.data_ptr(), n, cellp, sptr, c,
                                                  desc.data_ptr(), jac.data_ptr(), jac.shape[0], row_ptr.data_ptr(),
                                                  row_atom.data_ptr(), self._stream()))
        self.status()
        return Derivatives(desc, jac[:nrows], row_ptr, row_atom[:nrows])

    # ------------------------------------------------------------------ other output modes
    def coefficients(self, positions, numbers, cell=None, centers=None, out=None):
        """(C, W) expansion coefficients c^mu_nlm, W = S n_max (l_max+1)^2."""
        import torch
        n, c, cptr = self._inputs(positions, numbers, centers)
        keep, cellp = self._cell(cell)
        if out is None:
            out = torch.empty((c, self.n_coefficients), dtype=torch.float32, device=positions.device)
        self._check(self._lib.soap_coefficients(self._h, positions.data_ptr(), numbers.data_ptr(), n, cellp, cptr, c,
                                                out.data_ptr(), self._stream()))
        return out

    def coefficient_derivatives(self, positions, numbers, cell=None, centers=None) -> Derivatives:
        """Coefficients and their Jacobian in the row format of `derivatives` (width W)."""
        import torch
        _, nrows = self.neighbors(positions, numbers, cell, centers)
        n, c, cptr = self._inputs(positions, numbers, centers)
        keep, cellp = self._cell(cell)
        dev = positions.device
        coeff = torch.empty((c, self.n_coefficients), dtype=torch.float32, device=dev)
        jac = torch.empty((max(nrows, 1), 3, self.n_coefficients), dtype=torch.float32, device=dev)
        row_ptr = torch.empty(c + 1, dtype=torch.int64, device=dev)
        row_atom = torch.empty(max(nrows, 1), dtype=torch.int32, device=dev)
        self._check(self._lib.soap_coefficient_derivatives(self._h, positions.data_ptr(), numbers.data_ptr(), n, cellp, cptr, c,
                                                           coeff.data_ptr(), jac.data_ptr(), jac.shape[0], row_ptr.data_ptr(),
                                                           row_atom.data_ptr(), self._stream()))
        self.status()
        return Derivatives(coeff, jac[:nrows], row_ptr, row_atom[:nrows])

    def descriptor_average(self, mode, positions, numbers, cell=None, centers=None, out=None):
        """(F,) averaged descriptor, mode "inner" or "outer"."""
        import torch
        n, c, cptr = self._inputs(positions, numbers, centers)
        keep, cellp = self._cell(cell)
        if out is None:
            out = torch.empty(self.n_features, dtype=torch.float32, device=positions.device)
        self._check(self._lib.soap_descriptor_average(self._h, AVERAGE_MODES[mode], positions.data_ptr(), numbers.data_ptr(), n,
                                                      cellp, cptr, c, out.data_ptr(), self._stream()))
        return out

    def derivatives_average(self, mode, positions, numbers, cell=None, centers=None, out_desc=None, out_jac=None):
        """Averaged descriptor (F,) and its Jacobian (n_atoms, 3, F)."""
        import torch
        n, c, cptr = self._inputs(positions, numbers, centers)
        keep, cellp = self._cell(cell)
        if out_desc is None:
            out_desc = torch.empty(self.n_features, dtype=torch.float32, device=positions.device)
        if out_jac is None:
            out_jac = torch.empty((n, 3, self.n_features), dtype=torch.float32, device=positions.device)
        self._check(self._lib.soap_derivatives_average(self._h, AVERAGE_MODES[mode], positions.data_ptr(), numbers.data_ptr(), n,
                                                       cellp, cptr, c, out_desc.data_ptr(), out_jac.data_ptr(), self._stream()))
        return out_desc, out_jac

    def profile(self, enable=True):
        self._check(self._lib.soap_profile(self._h, int(bool(enable))))

    def profile_read(self):
        """(ms in the neighbour search, ms in the fused per-centre kernel) of the last call."""
        a, b = C.c_float(), C.c_float()
        self._check(self._lib.soap_profile_read(self._h, C.byref(a), C.byref(b)))
        return float(a.value), float(b.value)

    def derivatives_host(self, positions, numbers, cell, host_out, dev_buf, centers=None):
        """End-to-end call on HOST buffers: copies the (pinned) inputs to the device,
        computes, and copies descriptor, Jacobian, row_ptr and row_atom back into the
        pinned tensors of `host_out`.  `dev_buf` holds the device staging tensors.
        Everything is enqueued on the current stream; the caller synchronises."""
        dev_buf["pos"].copy_(positions, non_blocking=True)
        dev_buf["num"].copy_(numbers, non_blocking=True)
        self.derivatives_into(dev_buf["pos"], dev_buf["num"], cell, centers, dev_buf["desc"], dev_buf["jac"],
                              dev_buf["row_ptr"], dev_buf["row_atom"])
        for k in ("desc", "jac", "row_ptr", "row_atom"):
            host_out[k].copy_(dev_buf[k], non_blocking=True)

    def jacobian_dense(self, deriv, n_atoms=None, include=None, out=None):
        """(C, n_include, 3, F) dense Jacobian of a `Derivatives` result (zeros outside the spheres).
        `include` is an int32 device tensor of atom indices; without it atoms 0..n_atoms-1 are listed."""
        import torch
        c = deriv.row_ptr.shape[0] - 1
        if include is not None:
            assert include.is_cuda and include.dtype == torch.int32 and include.is_contiguous()
            n_inc, iptr = include.shape[0], C.c_void_p(include.data_ptr())
        else:
            n_inc, iptr = int(n_atoms), None
        width = deriv.jacobian.shape[2]                     # F, or W for the rows of the coefficient mode
        if out is None:
            out = torch.empty((c, n_inc, 3, width), dtype=torch.float32, device=deriv.jacobian.device)
        self._check(self._lib.soap_rows_dense(self._h, deriv.jacobian.data_ptr(), width, deriv.row_ptr.data_ptr(),
                                              deriv.row_atom.data_ptr(), c, iptr, n_inc, out.data_ptr(), self._stream()))
        return out

    def derivatives_batched(self, positions, numbers, cell=None, centers=None, batch=1024):
        """Yields (centre indices of the batch, Derivatives) for consecutive batches of centres, so that
        the Jacobian held on the device at any time is bounded by the batch (the paper's
        centre-batch streaming); `centers` defaults to all atoms."""
        import torch
        n = positions.shape[0]
        allc = torch.arange(n, dtype=torch.int32, device=positions.device) if centers is None else centers
        for lo in range(0, allc.shape[0], batch):
            part = allc[lo:lo + batch].contiguous()
            yield part, self.derivatives(positions, numbers, cell, part)

    def status(self):
        """Waits for the stream; raises if the device flagged a problem. Returns (n_pairs, n_rows)."""
        npairs, nrows = C.c_int64(), C.c_int64()
        self._check(self._lib.soap_status(self._h, C.byref(npairs), C.byref(nrows), self._stream()))
        return int(npairs.value), int(nrows.value)
