"""Drives ``rvh_steps`` for ALL ranks inside one process, in lock step: every rank's generator is
advanced to its next communication step, the step is carried out by plain copies (an exchange)
or a plain sum (an all-reduce), and so on.  The ranks' kernels are launched one after the other
on one stream and none waits for another, so the result is what separate processes compute."""
import torch

from paper_2006_02924_b200.rvh import AllReduce, Exchange, rvh_steps


def run_lockstep(size, xs, offsets, kernels):
    """xs[r] = rank r's gradient, kernels[r] = its arithmetic.  Returns the list of results."""
    gens = [rvh_steps(r, size, xs[r], offsets, kernels[r]) for r in range(size)]
    results = [None] * size
    log = []
    pending = []
    for r, g in enumerate(gens):
        try:
            pending.append(next(g))
        except StopIteration as done:
            results[r] = done.value
    while pending:
        assert len(pending) == size and len({type(p) for p in pending}) == 1, "ranks out of step"
        if isinstance(pending[0], Exchange):
            # all sends are read before any receive buffer of the SAME rank could alias them:
            # receive buffers never overlap what the rank sends in the same step
            staged = [p.send.clone() for p in pending]
            for r, p in enumerate(pending):
                assert pending[p.peer].peer == r, "exchange partners disagree"
                assert pending[p.peer].recv.numel() == p.send.numel()
                pending[p.peer].recv.copy_(staged[r])
            log.append(("exchange", [p.peer for p in pending], [p.send.numel() for p in pending]))
        else:
            assert isinstance(pending[0], AllReduce)
            seen = set()
            for r, p in enumerate(pending):
                if p.ranks in seen:
                    continue
                seen.add(p.ranks)
                assert r in p.ranks and all(pending[q].ranks == p.ranks for q in p.ranks)
                total = torch.stack([pending[q].tensor for q in p.ranks]).sum(dim=0)
                for q in p.ranks:
                    pending[q].tensor.copy_(total)
            log.append(("allreduce", sorted(seen)))
        nxt = []
        for r, g in enumerate(gens):
            try:
                nxt.append(next(g))
            except StopIteration as done:
                results[r] = done.value
        pending = nxt
    return results, log
