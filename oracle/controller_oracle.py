"""CPU oracle for the controller side of the streaming store.  TEST INFRASTRUCTURE ONLY.

Plain Python / numpy restatements of what the paper's TransferQueue controller does for one
request (Section 4.4 "Control Plane: Panoramic Data Admin" and its figure "Procedure for a get
request"), and of the load-balancing step it names there (one-dimensional bin packing solved
with the Karmarkar-Karp differencing method).  Nothing in the product path may import this
file; it shares no code with the CUDA library.

  put ......... a storage unit reports that some columns of some samples have been written:
                their status bits turn on (Section 4.2, last step of the interaction)
  get ......... build the mask of requested columns, find the samples whose requested columns
                are all ready and that this task has not been handed before, select the
                required number of them, record them as consumed, return their indices
  balance ..... split samples over k groups so that token totals are as even as possible;
                "DP" keeps the number of samples per group equal, "PP" drops that constraint

Readings where the paper is silent (of the selection it says only that the required number of
samples is chosen): eligible samples are taken in increasing global index; a request carries a
sample count and, optionally, a token budget; the selection is the longest prefix of the
eligible sequence within both limits, except that a first sample longer than the whole budget
is handed out alone.  Ties in the differencing method are broken as stated in kk_partition_ref.

Pins (tests/test_oracle_controller.py): brute-force definitions of eligibility and of the
longest admissible prefix; exactly-once consumption per task over repeated requests; the
two-way differencing method against its numbers-only form and the textbook example
{8,7,6,5,4} -> difference 2; brute-force optimum on tiny inputs as a lower bound; equal-size
and exact-cover properties.  No function here is "parity unpinned".
"""
from __future__ import annotations

import heapq

import numpy as np


# ----------------------------------------------------------------------------------------
# C1  put / get on the status table          (Section 4.4; Section 4.2 "Interaction Interface")
# ----------------------------------------------------------------------------------------
def controller_put_ref(ready: np.ndarray, idx, column_bits: int) -> None:
    """Mark the columns in ``column_bits`` of the samples in ``idx`` as written (in place)."""
    for i in idx:
        ready[int(i)] |= np.uint32(column_bits)


def controller_get_ref(ready: np.ndarray, consumed: np.ndarray, length, column_mask: int, task_bit: int,
                       max_samples: int, token_budget: int = 0):
    """One read request of RL task ``task_bit`` for the columns in ``column_mask``.

    ready[i]    : bit c set when column c of sample i has been written
    consumed[i] : bit t set when sample i has been handed to task t (updated in place)
    length[i]   : tokens of sample i (None: no lengths known; then token_budget must be <= 0)
    Returns (indices handed out, their token total, number of eligible samples seen).
    """
    n = ready.shape[0]
    chosen, tokens, eligible = [], 0, 0
    open_ = True                      # the prefix is still growing
    for i in range(n):
        if (int(ready[i]) & column_mask) != column_mask:
            continue                  # a requested column is not there yet
        if int(consumed[i]) & task_bit:
            continue                  # this task already got it
        eligible += 1
        if not open_:
            continue
        L = int(length[i]) if length is not None else 0
        fits = len(chosen) < max_samples and (token_budget <= 0 or tokens + L <= token_budget or not chosen)
        if fits:
            chosen.append(i)
            tokens += L
        else:
            open_ = False             # longest prefix: nothing after the first misfit
    for i in chosen:
        consumed[i] |= np.uint32(task_bit)
    return np.asarray(chosen, dtype=np.int32), tokens, eligible


# ----------------------------------------------------------------------------------------
# C2  Karmarkar-Karp balancing                     (Section 4.4, last paragraph; the method is
#     the largest differencing method of Karmarkar & Karp 1982 in its k-way form)
# ----------------------------------------------------------------------------------------
def kk_partition_ref(length, k: int, equal_size: bool):
    """Split items 0..n-1 with sizes ``length`` into k groups; returns part[i] in [0, k).

    State: partial solutions, each a list of k (sum, items) groups kept in decreasing order of
    sum; the spread of a partial solution is its largest minus its smallest sum.  Start with
    one partial solution per item (the item alone, k-1 empty groups); when ``equal_size`` is
    set, sort the items by decreasing size, cut them into consecutive runs of k (the last run
    padded with empty groups) and start with one partial solution per run, one item per group,
    so that every later merge adds the same number of items to every group.  Repeat: take the
    two partial solutions of largest spread and merge them, joining the j-th largest group of
    the first with the j-th smallest of the second; stop when one is left.

    Tie-breaks: items are ordered by (size descending, index ascending); partial solutions of
    equal spread are taken in order of creation; groups of equal sum keep their order
    (stable sort).  Group g of the result is the g-th largest sum.
    """
    length = [int(x) for x in length]
    n = len(length)
    order = sorted(range(n), key=lambda i: (-length[i], i))
    sols = []
    if equal_size:
        for s in range(0, n, k):
            run = order[s:s + k]
            sols.append([(length[i], [i]) for i in run] + [(0, []) for _ in range(k - len(run))])
    else:
        for i in order:
            sols.append([(length[i], [i])] + [(0, []) for _ in range(k - 1)])
    if not sols:
        return np.zeros(0, dtype=np.int32)
    heap = []
    for cid, sol in enumerate(sols):
        heapq.heappush(heap, (-(sol[0][0] - sol[-1][0]), cid, sol))
    next_id = len(sols)
    while len(heap) > 1:
        _, _, a = heapq.heappop(heap)
        _, _, b = heapq.heappop(heap)
        merged = [(a[j][0] + b[k - 1 - j][0], a[j][1] + b[k - 1 - j][1]) for j in range(k)]
        merged.sort(key=lambda g: -g[0])          # stable
        heapq.heappush(heap, (-(merged[0][0] - merged[-1][0]), next_id, merged))
        next_id += 1
    final = heap[0][2]
    part = np.zeros(n, dtype=np.int32)
    for g, (_, items) in enumerate(final):
        for i in items:
            part[i] = g
    return part


def group_sums(length, part, k: int) -> np.ndarray:
    """Token total of every group of a partition."""
    out = np.zeros(k, dtype=np.int64)
    for L, g in zip(length, part):
        out[int(g)] += int(L)
    return out
