"""CPU oracle for the fused equivariant message-passing convolution.

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain, fp64 statement of
what the CUDA path must compute.  It shares no code with the CUDA library or
its Python binding and must never be imported by the product path; only the
tests, the smoke check and the CPU-baseline / reference legs of the benchmark
may call it.

Modules
-------
cg    Clebsch-Gordan coefficients from the Racah closed form, the change to the
      real basis, the canonical sign, path enumeration, dense coupling tensor.
sh    Real spherical harmonics of any degree from the complex definition; of edge
      vectors (direction only) and their vector-Jacobian product by central
      differences in float64.
conv  Naive edge loops (plain C, fp64) for the convolution forward / backward
      and the standalone channelwise tensor product; on top of them, written
      from their definitions: padded edge lists, collapsed output
      multiplicities, the double backward, the radial network's last layer
      (s = h W in float64) and the convolution on edge vectors.
"""
