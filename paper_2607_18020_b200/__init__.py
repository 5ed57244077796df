"""B200-native fused finite-difference PDE-residual operators (forward residual + loss,
gather-form discrete adjoint, boundary-gradient correction) behind a C ABI.

    paper_2607_18020_b200.binding    ctypes binding of libfpde.so (fpde_fwd, fpde_bwd, ...)
    paper_2607_18020_b200.autograd   torch.autograd.Function wrappers over the binding
    paper_2607_18020_b200.workloads  seeded synthetic inputs (numpy only)
    paper_2607_18020_b200.build      builds libfpde.so in-tree with nvcc for sm_100a

Nothing is loaded at import time; the binding raises if the shared library is missing.
"""
__all__ = ["binding", "workloads", "build"]
