"""A small search driver built from the library's three device steps: decode -> evaluate -> select.

The paper solves the planning problem with a MIP and notes that heuristics for it are priority
dispatch rules (Section IV).  This module is such a heuristic in its simplest form, there to show
the three entry points working together on the device; it is not part of the evaluation path:

  population   K candidates, each an arbitrary priority list (a permutation of the operators)
               and an operator-to-machine assignment;
  generation   pe_decode_priority turns the lists into topological priority orders,
               pe_eval_batch scores them, the `elite` best feasible ones survive and the rest of
               the population is refilled with mutated copies of survivors (a few random rank
               swaps per list, a few reassigned operators per assignment);
  result       pe_select_best of the last generation, and the best candidate seen.

torch is used for the mutations (gather/scatter on the device) and for picking survivors;
the scheduling arithmetic is all in the library's kernels.
"""
import numpy as np


def evolve(graph, assign, lists, generations=20, elite=0.125, swaps=2, reassign=0, num_devices=None, seed=0,
           reject_mask=0xFFFFFFFF, flags=0):
    """graph: binding.Graph; assign: cuda uint8 [V, K]; lists: cuda int16 [V, K] (u16 operator ids per rank).
    Returns dict(best_makespan, best_assign [V], best_list [V], best_order [V], history [generations])."""
    import torch
    V, K = lists.shape
    dev = lists.device
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    n_elite = max(1, int(K * elite))
    big = torch.iinfo(torch.int32).max
    best = dict(best_makespan=big, history=[])
    cols = torch.arange(K, device=dev)
    for _ in range(generations):
        order, dstatus = graph.decode_priority(lists)
        out = graph.eval_batch(assign, order, flags=flags, want_times=False)
        bad = ((out["status"] & np.int32(np.uint32(reject_mask).view(np.int32))) != 0) | (dstatus != 0)
        score = torch.where(bad, torch.full_like(out["makespan"], big), out["makespan"])
        top = torch.argsort(score, stable=True)[:n_elite]
        gbest = int(score[top[0]])
        best["history"].append(gbest)
        if gbest < best["best_makespan"]:
            c = int(top[0])
            best.update(best_makespan=gbest, best_assign=assign[:, c].clone(), best_list=lists[:, c].clone(),
                        best_order=order[:, c].clone())
        # next generation: the elite unchanged, the rest mutated copies of random elite members
        parent = top[torch.randint(0, n_elite, (K,), device=dev, generator=gen)]
        parent[:n_elite] = top
        lists = lists[:, parent].contiguous()
        assign = assign[:, parent].contiguous()
        mut = cols >= n_elite
        for _s in range(swaps):
            r1 = torch.randint(0, V, (K,), device=dev, generator=gen)
            r2 = torch.randint(0, V, (K,), device=dev, generator=gen)
            r2 = torch.where(mut, r2, r1)                      # the elite keep their lists
            a, b = lists[r1, cols].clone(), lists[r2, cols].clone()
            lists[r1, cols] = b
            lists[r2, cols] = a
        for _s in range(reassign):
            i = torch.randint(0, V, (K,), device=dev, generator=gen)
            j = torch.randint(0, num_devices, (K,), device=dev, generator=gen).to(torch.uint8)
            assign[i, cols] = torch.where(mut, j, assign[i, cols])
    return best
