"""A face with the constructor keywords and call shapes of the paper's interface section.

`SOAP(r_cut=..., n_max=..., l_max=..., sigma=..., rbf="gto" | "polynomial", weighting=..., crossover=...,
average="off" | "inner" | "outer" | "cc", species=[...], periodic=...)`, `create()` (alias `generate()`)
returning one feature row per centre, `derivatives()` returning the dense (centres, atoms, 3, features)
array, an explicit list of centres (atom indices or Cartesian points) and an `include` / `exclude` atom
selection.  Argument marshalling only: every number comes from the CUDA library through `binding.Soap`.

A structure is anything with `positions` (N, 3), `numbers` (N,) and optionally `cell` (3, 3) and `pbc`
attributes (an ASE-like object), or a tuple `(positions, numbers[, cell])`.  Results are torch tensors on
the GPU.  Not offered: `sparse=True` output and the `max_num_neighbors` cap.
"""
from __future__ import annotations

import numpy as np

from .binding import GTO, POLYNOMIAL, Soap

_RBF = {"gto": GTO, "polynomial": POLYNOMIAL}


class SOAP:
    def __init__(self, r_cut, n_max, l_max, sigma=1.0, rbf="gto", weighting=None, crossover=True, average="off",
                 species=None, periodic=False, sparse=False, device="cuda", quad_n=None, max_num_neighbors=None):
        if species is None:
            raise ValueError("species must be given")
        if sparse:
            raise NotImplementedError("sparse output is not offered")
        if max_num_neighbors is not None:
            raise NotImplementedError("a cap on the neighbour count is not offered")
        if average not in ("off", "inner", "outer", "cc"):
            raise ValueError("average must be 'off', 'inner', 'outer' or 'cc'")
        if rbf not in _RBF:
            raise ValueError("rbf must be 'gto' or 'polynomial'")
        if not str(device).startswith("cuda"):
            raise ValueError("this library runs on a CUDA device only")
        # quad_n steers the paper's on-device quadrature; here the radial integrals are tabulated once on the
        # host to fp32 rounding, so the argument is accepted and has nothing to steer
        self.average = average
        self.periodic = bool(periodic)
        self._args = dict(species=[_z(z) for z in species], r_cut=float(r_cut), n_max=int(n_max), l_max=int(l_max),
                          sigma=float(sigma), rbf=_RBF[rbf], crossover=bool(crossover), weighting=weighting)
        self._soap = {}                                     # one library object per periodicity pattern

    # ------------------------------------------------------------------ plumbing
    def _engine(self, pbc):
        if pbc not in self._soap:
            self._soap[pbc] = Soap(pbc=pbc, **self._args)
        return self._soap[pbc]

    def _unpack(self, system):
        import torch
        if isinstance(system, (tuple, list)):
            positions, numbers = system[0], system[1]
            cell = system[2] if len(system) > 2 else None
            pbc = None
        else:
            positions, numbers = system.positions, system.numbers
            cell = getattr(system, "cell", None)
            pbc = getattr(system, "pbc", None)
        if cell is not None:
            cell = np.asarray(cell, np.float64).reshape(3, 3)
            if not np.any(cell):
                cell = None
        if pbc is None:
            pbc = (self.periodic,) * 3
        pbc = tuple(bool(p) and self.periodic for p in np.broadcast_to(np.asarray(pbc, bool), (3,)))
        if any(pbc) and cell is None:
            raise ValueError("a periodic structure needs a cell")
        pos = torch.as_tensor(np.ascontiguousarray(positions, np.float32) if not torch.is_tensor(positions) else positions)
        num = torch.as_tensor(np.ascontiguousarray(numbers, np.int32) if not torch.is_tensor(numbers) else numbers)
        return pos.to("cuda", torch.float32).contiguous(), num.to("cuda", torch.int32).contiguous(), cell, pbc

    @staticmethod
    def _centers(centers, device):
        """None, a list of atom indices, or an array of Cartesian points (C, 3)."""
        import torch
        if centers is None:
            return None, None
        arr = centers.detach().cpu().numpy() if torch.is_tensor(centers) else np.asarray(centers)
        if arr.ndim == 2 and arr.shape[1] == 3 and not np.issubdtype(arr.dtype, np.integer):
            return None, torch.as_tensor(np.ascontiguousarray(arr, np.float32)).to(device)
        return torch.as_tensor(np.ascontiguousarray(arr.reshape(-1), np.int32)).to(device), None

    def get_number_of_features(self):
        e = self._engine((False, False, False))
        return e.n_coefficients if self.average == "cc" else e.n_features

    # ------------------------------------------------------------------ lists of structures
    @staticmethod
    def _is_list_of_systems(system):
        if not isinstance(system, (list, tuple)) or len(system) == 0:
            return False
        first = system[0]
        return hasattr(first, "positions") or (isinstance(first, (list, tuple)) and len(first) >= 2 and np.ndim(first[0]) == 2)

    def _many(self, systems, derivatives):
        """Non-periodic structures, every atom a centre, average 'off': one batch call for all of them."""
        import torch
        from .binding import Derivatives
        parts = [self._unpack(s) for s in systems]
        if self.average != "off" or any(any(p[3]) for p in parts):
            return None
        e = self._engine((False, False, False))
        sizes = [p[0].shape[0] for p in parts]
        pos = torch.cat([p[0] for p in parts]).contiguous()
        num = torch.cat([p[1] for p in parts]).contiguous()
        ptr = torch.tensor(np.concatenate([[0], np.cumsum(sizes)]), dtype=torch.int64, device=pos.device)
        if not derivatives:
            d = e.derivatives_batch(pos, num, ptr, jacobian=False)
            return list(torch.split(d, sizes))
        out = e.derivatives_batch(pos, num, ptr)
        row_ptr = out.row_ptr
        res, a = [], 0
        for n in sizes:
            r0, r1 = int(row_ptr[a]), int(row_ptr[a + n])
            one = Derivatives(out.descriptor[a:a + n], out.jacobian[r0:r1], (row_ptr[a:a + n + 1] - r0).contiguous(),
                              (out.row_atom[r0:r1] - a).contiguous())
            res.append((e.jacobian_dense(one, n_atoms=n) if n else out.jacobian.new_zeros((0, 0, 3, e.n_features)), one.descriptor))
            a += n
        e.status()
        return res

    # ------------------------------------------------------------------ descriptors
    def create(self, system, centers=None):
        """(n_centres, n_features); one row, (1, n_features), for the inner and outer averages.  A list of
        structures gives a list of results (non-periodic structures with every atom a centre go through one
        batch call)."""
        if self._is_list_of_systems(system):
            if centers is None:
                many = self._many(system, False)
                if many is not None:
                    return many
            return [self.create(s, None if centers is None else centers[k]) for k, s in enumerate(system)]
        pos, num, cell, pbc = self._unpack(system)
        e = self._engine(pbc)
        idx, sites = self._centers(centers, pos.device)
        if sites is not None:
            if self.average != "off":
                raise NotImplementedError("centres at arbitrary points are offered for average='off' only")
            return e.derivatives_at(pos, num, sites, cell, jacobian=False)
        if self.average == "off":
            out = e.descriptor(pos, num, cell, idx)
        elif self.average == "cc":
            out = e.coefficients(pos, num, cell, idx)
        else:
            out = e.descriptor_average(self.average, pos, num, cell, idx)[None]
        e.status()
        return out

    generate = create

    # ------------------------------------------------------------------ derivatives
    def derivatives(self, system, centers=None, include=None, exclude=None, return_descriptor=True):
        """Dense derivatives (n_centres, n_included_atoms, 3, n_features) — zeros for atoms outside a centre's
        sphere — and, with return_descriptor, the descriptor; (1, n_included_atoms, 3, n_features) for the
        averages.  `include` / `exclude` select the atoms to differentiate with respect to."""
        import torch
        if include is not None and exclude is not None:
            raise ValueError("give include or exclude, not both")
        if self._is_list_of_systems(system):
            many = self._many(system, True) if centers is None and include is None and exclude is None else None
            if many is None:
                many = [self.derivatives(s, None if centers is None else centers[k], include, exclude, True)
                        for k, s in enumerate(system)]
            return many if return_descriptor else [m[0] for m in many]
        pos, num, cell, pbc = self._unpack(system)
        n = pos.shape[0]
        e = self._engine(pbc)
        if exclude is not None:
            include = np.setdiff1d(np.arange(n), np.asarray(exclude, np.int64))
        inc = None if include is None else torch.as_tensor(np.ascontiguousarray(np.asarray(include).reshape(-1), np.int32)).to(pos.device)
        idx, sites = self._centers(centers, pos.device)
        if self.average in ("inner", "outer"):
            if sites is not None:
                raise NotImplementedError("centres at arbitrary points are offered for average='off' only")
            desc, jac = e.derivatives_average(self.average, pos, num, cell, idx)
            e.status()
            jac = jac if inc is None else jac[inc.long()]
            return (jac[None], desc[None]) if return_descriptor else jac[None]
        if sites is not None:
            if self.average != "off":
                raise NotImplementedError("centres at arbitrary points are offered for average='off' only")
            d = e.derivatives_at(pos, num, sites, cell)
        elif self.average == "cc":
            d = e.coefficient_derivatives(pos, num, cell, idx)
        else:
            d = e.derivatives(pos, num, cell, idx)
        dense = e.jacobian_dense(d, n_atoms=n, include=inc)
        e.status()
        return (dense, d.descriptor) if return_descriptor else dense


def _z(z):
    """Atomic number from a number or a chemical symbol of the first three periods and a few more."""
    if isinstance(z, str):
        table = ["H", "He", "Li", "Be", "B", "C", "N", "O", "F", "Ne", "Na", "Mg", "Al", "Si", "P", "S", "Cl", "Ar",
                 "K", "Ca", "Sc", "Ti", "V", "Cr", "Mn", "Fe", "Co", "Ni", "Cu", "Zn", "Ga", "Ge", "As", "Se", "Br", "Kr"]
        return table.index(z) + 1
    return int(z)
