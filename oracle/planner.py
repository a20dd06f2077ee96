"""Oracle: bit-width-aware I/O-compute pipeline planning (Section 3.4).  Test infrastructure only.

With the nested store an expert requested at several widths is loaded segment by segment: segment k
holds what width bits[k] adds to width bits[k-1], and a request at width index k needs segments 0..k
(Section 3.4: "all three requests call the INT2 weight ... the two requests requiring INT3 further
call the medium blue weight").  Per layer, B[j][k] counts the requests of expert j at width index k
(the matrix B_{j,k} of Section 3.4.3).

* ``load_items``: what has to be loaded: for every expert with a request, segments 0..(its largest
  requested width index), ascending.
* ``hebf_order`` (Hottest-Expert-Bit-First, the three steps printed under "Solution"): one queue per
  expert in ascending width; repeatedly take, among the queue heads, the item with the highest
  frequency.  Reading: the frequency of item (j, k) is the number of requests that read segment k of
  expert j, sum over k' >= k of B[j][k'] (the reuse count of the paper's own example); ties go to the
  lower expert id (the order of the sequential baseline).
* ``id_order``: the sequential baseline of Fig. 9(b, c): ascending expert id, ascending width.
* ``simulate``: the two-queue pipeline of Eq. 6.  Loads run back to back in queue order, item s taking
  T_io[k_s]; the compute of item s (its B[j][k] requests, each T_comp[k]) starts when both its load
  (constraint 6a) and the compute of item s-1 have finished; the time it stood idle before starting is
  T_wait of constraint 6c.  Returns the makespan and the summed wait.
* ``budget_step`` (Algorithm 2, one layer): the segments a layer needs are loaded into a memory budget
  M; when they do not fit, resident segments of other layers are released, highest width first
  ("high bit-width expert weights are released ... low bit-width weights are also released as
  needed"), oldest layer first among equal widths, until the layer fits.  Reading: the printed loop
  frees "layer[j-1][k]" for k = 0..K-1 and then "[1]"; the text next to it fixes the order (high
  widths before low ones), which is what is written out here.  PARITY UNPINNED beyond that text.
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple

Item = Tuple[int, int]          # (expert, segment / width index)


def load_items(B: Sequence[Sequence[int]]) -> Dict[int, List[Item]]:
    out: Dict[int, List[Item]] = {}
    for j, row in enumerate(B):
        ks = [k for k, n in enumerate(row) if n > 0]
        if ks:
            out[j] = [(j, k) for k in range(max(ks) + 1)]
    return out


def frequency(B: Sequence[Sequence[int]], item: Item) -> int:
    j, k = item
    return sum(B[j][k:])


def id_order(B: Sequence[Sequence[int]]) -> List[Item]:
    q = load_items(B)
    return [it for j in sorted(q) for it in q[j]]


def hebf_order(B: Sequence[Sequence[int]]) -> List[Item]:
    queues = load_items(B)
    heads = {j: 0 for j in queues}
    out: List[Item] = []
    while heads:
        best = None
        for j in sorted(heads):
            it = queues[j][heads[j]]
            if best is None or frequency(B, it) > frequency(B, best):
                best = it
        out.append(best)
        j = best[0]
        heads[j] += 1
        if heads[j] == len(queues[j]):
            del heads[j]
    return out


def simulate(B: Sequence[Sequence[int]], order: Sequence[Item], t_io: Sequence[float],
             t_comp: Sequence[float]) -> Tuple[float, float]:
    load_end = 0.0
    comp_end = 0.0
    wait = 0.0
    seen = set()
    for j, k in order:
        assert (j, k) not in seen and (k == 0 or (j, k - 1) in seen), "ascending width per expert (constraint 6b)"
        seen.add((j, k))
        load_end += t_io[k]
        n = B[j][k]
        if n > 0:
            start = max(comp_end, load_end)
            wait += start - comp_end
            comp_end = start + n * t_comp[k]
    return max(comp_end, load_end), wait


def budget_step(resident: List[Tuple[int, int, int, int]], need: Sequence[Tuple[int, int, int, int]],
                budget: int) -> Tuple[List[Tuple[int, int, int, int]], List[Tuple[int, int, int, int]],
                                      List[Tuple[int, int, int, int]]]:
    """resident / need: (layer, expert, segment, bytes).  Returns (new resident list, loads, evictions).
    Segments of `need` already resident are kept; the rest are loaded after enough other segments have been
    released, highest segment index first, then oldest layer, then lowest expert id."""
    have = {(l, e, k) for l, e, k, _ in resident}
    needed = {(l, e, k) for l, e, k, _ in need}
    loads = [x for x in need if (x[0], x[1], x[2]) not in have]
    used = sum(b for _, _, _, b in resident)
    want = sum(b for _, _, _, b in loads)
    evict: List[Tuple[int, int, int, int]] = []
    if used + want > budget:
        victims = sorted((x for x in resident if (x[0], x[1], x[2]) not in needed),
                         key=lambda x: (-x[2], x[0], x[1]))
        for v in victims:
            if used + want <= budget:
                break
            evict.append(v)
            used -= v[3]
    assert used + want <= budget, "the layer's own segments exceed the budget"
    gone = {(l, e, k) for l, e, k, _ in evict}
    new_res = [x for x in resident if (x[0], x[1], x[2]) not in gone] + list(loads)
    return new_res, loads, evict
