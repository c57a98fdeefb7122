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
  result       the best candidate seen.

`evolve` mutates lists and assignments directly; `evolve_keys` is the biased random-key variant for fixed
assignments (a candidate is a vector of keys, its priority list their argsort).

torch is used for the mutations (gather/scatter on the device) only; decoding, the scheduling arithmetic
and the choice of the survivors (pe_select_topk, pe_select_best) are all in the library's kernels.
"""
import numpy as np


def _elite(graph, out, n, reject_mask):
    """The elite of a generation through the library's selection steps: the n best qualifying candidates
    (pe_select_topk; padded by repeating the first one when fewer qualify, or by candidate 0 when none does)
    and the best of all (pe_select_best).  Returns (elite indices [n], how many qualify, best index, its
    makespan or INT32_MAX)."""
    import torch
    idx, cnt = graph.select_topk(out, n, reject_mask)
    c, mk, _ = graph.select_best(out, reject_mask)
    n_ok = int(cnt.item())
    idx = idx.to(torch.int64)
    if n_ok < n:
        idx = torch.where(torch.arange(n, device=idx.device) < n_ok, idx, idx[0].clamp(min=0))
    return idx, n_ok, max(c, 0), (mk if c >= 0 else torch.iinfo(torch.int32).max)


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
        out["status"] |= dstatus                               # a list that is not a permutation is no candidate
        top, n_ok, c, gbest = _elite(graph, out, n_elite, reject_mask)
        best["history"].append(gbest)
        if gbest < best["best_makespan"]:
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


def evolve_keys(graph, assign, generations=200, elite=0.1, mutants=0.2, bias=0.7, seed=0, reject_mask=0xFFFFFFFF,
                flags=0):
    """Biased random-key search over priority lists for fixed assignments (the random-key encoding of
    sequencing problems: a candidate is a vector of keys in [0, 1), its priority list their argsort).
    Each generation keeps the `elite` best, replaces the `mutants` worst by fresh random keys and fills
    the rest by uniform crossover of an elite parent (each key taken with probability `bias`) with any
    other candidate.  graph: binding.Graph; assign: cuda uint8 [V, K], column c is candidate c's assignment
    throughout.  Returns dict(best_makespan, best_order [V], history)."""
    import torch
    V, K = assign.shape
    dev = assign.device
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    n_el, n_mut = max(2, int(K * elite)), int(K * mutants)
    big = torch.iinfo(torch.int32).max
    mask_bits = int(np.uint32(reject_mask).view(np.int32))
    keys = torch.rand((V, K), device=dev, generator=gen)
    best = dict(best_makespan=big, history=[])
    for _ in range(generations):
        lists = torch.argsort(keys, dim=0).to(torch.int16).contiguous()
        order, dstatus = graph.decode_priority(lists)
        out = graph.eval_batch(assign, order, flags=flags, want_times=False)
        out["status"] |= dstatus
        top, n_ok, c, gbest = _elite(graph, out, n_el, reject_mask)
        best["history"].append(gbest)
        if gbest < best["best_makespan"]:
            best.update(best_makespan=gbest, best_order=order[:, c].clone(), best_column=c)
        pa = top[torch.randint(0, n_el, (K,), device=dev, generator=gen)]
        pb = torch.randint(0, K, (K,), device=dev, generator=gen)
        take = torch.rand((V, K), device=dev, generator=gen) < bias
        child = torch.where(take, keys[:, pa], keys[:, pb])
        child[:, :n_el] = keys[:, top]
        if n_mut:
            child[:, K - n_mut:] = torch.rand((V, n_mut), device=dev, generator=gen)
        keys = child
    return best
