"""Batched Sailor plan simulator and plan search for NVIDIA B200 (sm_100a).

The computation lives in ``libsailor_b200.so`` (CUDA, built in-tree by ``build.py``) behind the
C ABI of ``include/sailor.h``.  ``binding`` exposes the same entry points to Python and only
marshals arguments; ``workloads`` generates seeded synthetic inputs; ``sharding`` splits one
search space over several GPUs.  Nothing here computes a plan on the CPU: without the CUDA
library, ``binding.load()`` raises.

    from paper_2504_17096_b200 import binding as B, workloads as W
    w = W.config2()
    ctx = B.sailor_create(w, device=0, stream=0)
    B.sailor_set_availability(ctx, w.avail)
    best, stats = B.sailor_plan(ctx, B.make_space(w), B.make_objective(w), k=8)
    B.sailor_destroy(ctx)
"""

__all__ = ["binding", "build", "sharding", "workloads"]
