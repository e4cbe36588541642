"""B200-native physics loss for data-free generative PDE solvers.

``inputs``  -- seeded synthetic workloads (numpy only, no method arithmetic).
``binding`` -- thin ctypes binding of the C-ABI CUDA library (``libdn.so``):
               ``dn_kl_field``, ``dn_energy``, ``dn_energy_grad``, ``dn_apply_bc``.
``autograd`` -- the loss as a differentiable PyTorch op (backward = the kernel's residual).
``sharding`` -- batch split across ranks by the paper's data-parallel rule.

The binding is imported on first attribute access so that the input generators
can be used without the CUDA library being built.
"""
import importlib

__all__ = ["inputs", "binding", "autograd", "sharding"]


def __getattr__(name):
    if name in ("binding", "inputs", "build", "autograd", "sharding"):
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
