"""RoutePack planner hot path for B200 (sm_100a): C-ABI CUDA library + thin binding.

``windows``  seeded synthetic optimizer-step windows (inputs only)
``build``    compiles ``csrc/*.cu`` into ``librp_b200.so`` with nvcc
``binding``  ctypes marshalling of the ``rp_*`` entry points declared in ``include/routepack.h``

Importing the package loads nothing; the CUDA library is opened on first use and every
call fails loudly if it is missing (there is no CPU path).
"""
__all__ = ["windows", "build", "binding"]
