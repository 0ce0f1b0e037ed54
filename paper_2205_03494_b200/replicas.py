"""Aggregation of client replicas that live on several GPUs (Sec. 1: the clients' models are sent
back and aggregated; Sec. 2.5: every client compresses its own subset).

Plumbing only: the library calls do the arithmetic on each GPU (omc_aggregate_sum adds up the
GPU's own clients, omc_aggregate_add those beyond the first sixteen, omc_divide turns the total
into the mean); in between, one all-reduce of
``torch.distributed`` adds the per-GPU sums and another the client counts.  Every buffer handed to
the collective is owned by the calling rank; no kernel of the library ever sees another GPU's
memory.  The two steps are passed in as callables so that the bookkeeping can be run on CPU ranks
(``gloo``) with stand-ins.
"""
from __future__ import annotations


def mean_across_ranks(out, n_local_clients: int, local_sum, divide, group=None):
    """``out`` (a tensor in the plan's full layout, owned by this rank) receives the mean over the
    clients of all ranks.

    local_sum(out)        writes the un-divided FP32 sum of this rank's clients into ``out``
                          (omc_aggregate_sum); a rank without clients passes n_local_clients = 0
                          and its callable must fill ``out`` with zeros.
    divide(out, k_total)  divides ``out`` by the total number of clients (omc_divide).
    Returns k_total.  The per-rank sums are added by the collective in an order it does not
    define, so with three or more ranks the last bits may differ from a single-GPU omc_aggregate.
    """
    import torch
    import torch.distributed as dist
    if n_local_clients < 0:
        raise ValueError("n_local_clients must not be negative")
    local_sum(out)
    count = torch.tensor([n_local_clients], dtype=torch.int64, device=out.device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(count, op=dist.ReduceOp.SUM, group=group)
        dist.all_reduce(out, op=dist.ReduceOp.SUM, group=group)
    k_total = int(count.item())
    if k_total <= 0:
        raise ValueError("no client on any rank")
    divide(out, k_total)
    return k_total


def mean_of_local_and_remote_clients(plans, packed, resid, sb, out, stream=0, group=None, layout_plan=None):
    """The GPU form: this rank's clients are (plans[k], packed[k], resid[k], sb[k]) as for
    ``aggregate``; ``out`` is a CUDA tensor in the plan's full layout.  A rank without clients
    passes empty lists and ``layout_plan``, any prepared plan of the same variables."""
    import paper_2205_03494_b200 as omc
    layout_plan = plans[0] if plans else layout_plan

    def local_sum(t):
        # any number of clients: the first batch starts the sum, each further batch is added to it,
        # in client order throughout
        if not plans:
            t.zero_()
        step = omc.MAX_CLIENTS_PER_CALL
        for a in range(0, len(plans), step):
            call = omc.aggregate_sum if a == 0 else omc.aggregate_add
            call(plans[a:a + step], packed[a:a + step], resid[a:a + step], sb[a:a + step], t.data_ptr(), stream)

    return mean_across_ranks(out, len(plans), local_sum,
                             lambda t, k: omc.divide(layout_plan, t.data_ptr(), k, stream), group)
