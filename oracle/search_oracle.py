"""CPU oracle of the two configuration searches.  TEST INFRASTRUCTURE, not product code.

Bisection search (Algorithm 1) and greedy search (Algorithm 2) of the paper, written step by
step over an abstract `evaluate(config) -> accuracy` callable.  Shares no code with the CUDA
path's host drivers.

Readings where the pseudo-code is silent or loose:
  * `for b in bs`: the working configuration starts at max(bs), so the loop visits the
    remaining bit widths from high to low (the text: the highest quantized precision first,
    then each lower one).
  * the halving steps use integer floor division;
  * Algorithm 1 ends its inner loop when the threshold stops changing and then writes b to
    ll[0:thr] even if the last evaluation at thr failed; here the largest prefix KNOWN to meet
    the target (lowl) is written instead, so the returned configuration always met the target
    when it was evaluated (or was never lowered).
"""
from __future__ import annotations

from typing import Callable, List, Sequence, Tuple


def bisection_search(n_layers: int, order: Sequence[int], bs: Sequence[int], target: float,
                     evaluate: Callable[[List[int]], float]) -> Tuple[List[int], List[List[int]]]:
    """Algorithm 1.  `order` lists the layers by ascending sensitivity.  Returns the final working
    configuration and the list of configurations evaluated, in order."""
    top = max(bs)
    w = [top] * n_layers                      # initialise working configuration with max(bs)
    ll = list(order)                          # layer list, sorted by sensitivity
    visited = []
    for b in sorted((v for v in bs if v != top), reverse=True):
        thr = len(ll) // 2
        upl = len(ll)
        lowl = 0
        while True:
            lw = list(w)                      # local working configuration
            for l in ll[:thr]:
                lw[l] = b
            a = evaluate(lw)
            visited.append(lw)
            old = thr
            if a >= target:
                lowl = thr
                thr = thr + (upl - thr) // 2
            else:
                upl = thr
                thr = thr - (thr - lowl) // 2
            if thr == old:
                break
        for l in ll[:lowl]:
            w[l] = b
        ll = ll[:lowl]                        # reduce the layer list for the next bit width
    return w, visited


def greedy_search(n_layers: int, order: Sequence[int], bs: Sequence[int], target: float,
                  evaluate: Callable[[List[int]], float]) -> Tuple[List[int], List[List[int]]]:
    """Algorithm 2.  Returns the final working configuration and the configurations evaluated."""
    top = max(bs)
    w = [top] * n_layers
    ll = list(order)
    visited = []
    for b in sorted((v for v in bs if v != top), reverse=True):
        ql = []                               # layers that took bit width b
        for l in ll:
            last = w[l]
            w[l] = b
            a = evaluate(list(w))
            visited.append(list(w))
            if a >= target:
                ql.append(l)
            else:
                w[l] = last                   # back to the last working value
        ll = ql
    return w, visited
