"""B200-native SPDP decode path: Tiled-CBC packing and dynamically pruned spMspV.

`paper_2607_21985_b200.spdp` is the Python binding of the C-ABI library (include/spdp.h);
`paper_2607_21985_b200.workloads` holds the seeded synthetic input generators.  Importing the
package loads nothing; the binding loads the CUDA library on first use and raises if it is
missing (there is no CPU fallback).
"""
