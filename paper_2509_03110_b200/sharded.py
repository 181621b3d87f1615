"""Workers sharded over several GPUs: one context per rank, one exchange per sync.

Algorithm 2 runs one worker per device.  Here every rank holds K of the K_total workers as stacked [K, d] tensors;
between syncs the ranks do not talk.  When the sync trigger fires, the sum over ALL workers of their iterate
accumulators is the only quantity the centre update needs: it is all-reduced in place, and every rank then applies
the same centre update, so the centres stay identical without a broadcast.  The schedule is keyed by the global
worker index, so the sharded run replays the run of one context that holds all K_total workers.

The exchange is argument plumbing around `torch.distributed.all_reduce`; the arithmetic stays in the library.
"""
import torch.distributed as dist


def shard_range(K_total, rank, world):
    """Workers [k_offset, k_offset + K) of rank `rank`: equal shards, K_total must divide by the world size."""
    if K_total % world != 0:
        raise ValueError(f"K_total = {K_total} workers do not divide over {world} ranks")
    K = K_total // world
    return rank * K, K


def exchange_and_couple(engine, group=None):
    """Sum the iterate accumulators of all ranks into every rank's accumulator, then run the sync branch.

    `engine` exposes acc_tensor() (the accumulator as a tensor that aliases the engine's own buffer), couple(), and
    optionally `stream` (a torch CUDA stream the engine's kernels run on).  Call it on every rank when
    engine.should_couple() holds; in the lock-step schedule that is the same tick on every rank.
    """
    acc = engine.acc_tensor()
    stream = getattr(engine, "stream", None)
    if acc.is_cuda and stream is not None:
        import torch

        # the collective is ordered after the ticks already enqueued on the engine's stream, and the centre update after it
        with torch.cuda.stream(stream):
            dist.all_reduce(acc, op=dist.ReduceOp.SUM, group=group)
    else:
        dist.all_reduce(acc, op=dist.ReduceOp.SUM, group=group)
    return engine.couple()
