"""Replicas of the whole model on several GPUs (Sec. 5): every rank trains its own copy on its own shard and the
copies are synchronised infrequently, at the end of an epoch, by averaging the parameters in place."""


def average_across_ranks(tensors, group=None):
    """All-reduce (sum) every tensor in place and divide by the number of ranks.  tensors: iterable of torch tensors
    (for an Engine: engine.param_tensors().values(), which alias the device arrays, so nothing is copied; with the
    NCCL backend the reduction runs over NVLink).  Without an initialised process group this is a no-op."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return 1
    world = dist.get_world_size(group)
    if world == 1:
        return 1
    work = [dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group, async_op=True) for t in tensors]
    for w in work:
        w.wait()
    for t in tensors:
        t.div_(world)
    return world
