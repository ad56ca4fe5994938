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
    space = B.make_space(w)
    best, stats = B.sailor_plan(ctx, space, B.make_objective(w), k=8)          # best plans of the segment space
    pruned, _ = B.sailor_plan(ctx, space, B.make_objective(w, flags=B.FLAG_DEGREE_ORDER), k=8)   # with H3/H4
    dp, dp_stats = B.sailor_plan_dp(ctx, space, B.all_zone_orders(w.n_zones), k=8)  # a GPU type per stage (Eq. 1)
    t, mem, cost, status = B.sailor_simulate(ctx, B.pack_records(W.random_plans(w, 1000, seed=1)))
    mixed = B.pack_mixed_plans(W.random_mixed_plans(w, 1000, seed=1))               # replicas of unlike types
    t, mem, cost, status = B.sailor_simulate_mixed(ctx, mixed)
    B.sailor_destroy(ctx)
"""

__all__ = ["binding", "build", "sharding", "workloads"]
