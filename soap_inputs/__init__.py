"""Seeded synthetic atomic structures shaped like the paper's workloads.

This module only draws coordinates and species.  It holds none of the SOAP
arithmetic, so both the CPU oracle's tests and the CUDA path's tests and
benchmark may import it.  Every structure is a pure function of its arguments
(NumPy PCG64 stream, `Generator.random` only) and positions are returned in
fp32, the precision the library takes its inputs in.

The paper benchmarks on water clusters (H2O)_n (Results section) but prints
neither coordinates nor a generator; the recipes below are stand-ins:

* `water_cluster(n_mol, seed)`: O sites uniform in a sphere at
  0.0334 molecules/A^3, rejected when any O-O distance is below 2.5 A; rigid
  molecules with r(OH) = 0.9572 A, angle(HOH) = 104.52 deg and a uniformly
  random orientation; atom order O, H, H per molecule.
* `multispecies_box(n_atoms, seed)`: C:H:N:O = 3:5:1:1 shuffled, uniform in a
  cubic periodic cell at 0.1 atoms/A^3 with minimum-image pair distance of at
  least 0.9 A.
* `small_periodic_cell(seed)`: 8 atoms in a 4 A triclinic cell, so that
  several periodic images of one atom fall inside a cutoff sphere.
"""
from .structures import (Structure, water_cluster, multispecies_box,
                         small_periodic_cell, random_rotation)

__all__ = ["Structure", "water_cluster", "multispecies_box",
           "small_periodic_cell", "random_rotation"]
