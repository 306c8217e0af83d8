"""libgmlp for B200 (sm_100a): the fused Gated MLP  Y = (SiLU(X Wg) * (X Wu)) Wd  with an
optional RMSNorm prologue, as hand-written CUDA kernels behind a C ABI.

``paper_2606_26344_b200.gmlp`` is the thin ctypes binding over ``libgmlp.so``;
``paper_2606_26344_b200.inputs`` holds the seeded synthetic workloads.  Importing the
package does not load the CUDA library; the first use of the binding does, and fails
loudly if the library has not been built.
"""
__all__ = ["gmlp", "inputs"]
