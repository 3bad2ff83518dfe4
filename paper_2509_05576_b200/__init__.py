"""B200-native per-layer quantizer (sensitivity-ordered, row-parallel, shared inverse Hessian).

``paper_2509_05576_b200.ptq`` is the thin binding over the C-ABI CUDA library;
``paper_2509_05576_b200.workloads`` draws the seeded synthetic layers.  Importing the
package itself loads neither torch nor the CUDA library.
"""
__all__ = ["ptq", "workloads"]
