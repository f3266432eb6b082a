"""Call order of one step on N replicas (one process per GPU, `torch.distributed` for the exchange).

Two ways of spreading Eq. (1) over replicas, both without any weight traffic: every replica holds all masters and
applies the same update, so the masters stay bit-identical.

batch-sharded (the default): every replica evaluates the SAME direction on its own shard of the mini-batch; one
all-reduce of (sum L+, sum L-, labelled positions) - three doubles, 24 bytes - gives everyone the full-batch losses,
hence the same g and the same Eq. (2).

direction-parallel (Eq. (1) with q = number of replicas): every replica evaluates its OWN direction (seed + rank) on
the same batch; an all-gather of the q update factors fl((lr / q) g_i) - 4 bytes each - and everyone applies all q
updates in rank order in one pass over the masters.

Only the order of library calls and collectives lives here; `model` is a binding.ZoqatModel (or anything with the same
methods) and `dist` is torch.distributed (or a stand-in with all_reduce / all_gather_into_tensor).
"""


def batch_sharded_step(model, dist, world, tokens, labels, seed, eps, lr, sums, result, rates=None):
    """rates: (lr_quant, lr_smooth) for models with Section 4.2 parameters (those move at once; the weights' update
    rides on the next step like everyone's)."""
    model.zoqat_step_begin(tokens, labels, seed, eps, sums)
    if world > 1:
        dist.all_reduce(sums)
    if rates is not None:
        model.zoqat_step_finish_rates_deferred(sums, seed, eps, lr, rates[0], rates[1], result)
    else:
        model.zoqat_step_finish_deferred(sums, seed, eps, lr, result)
    return result


def direction_parallel_step(model, dist, rank, world, tokens, labels, seed, eps, lr, sums, result, scales):
    """scales: float32 tensor [world] on the device of `result`; direction i = seed + i belongs to rank i."""
    model.zoqat_step_begin(tokens, labels, seed + rank, eps, sums)
    # the factor of Eq. (2) for one of q directions: fl(fl(lr / q) * g_i); lr / q is a binary32 division (the double
    # quotient of two binary32 values rounds to it)
    model.zoqat_step_result(sums, eps, lr_over_q(lr, world), result)
    mine = result[3:4]                                    # update_scale of this replica's direction
    if world > 1:
        dist.all_gather_into_tensor(scales, mine)
    else:
        scales.copy_(mine)
    model.zoqat_apply_update_multi([seed + i for i in range(world)], scales)
    return result


def lr_over_q(lr, q):
    import struct
    lr32 = struct.unpack("f", struct.pack("f", lr))[0]
    return struct.unpack("f", struct.pack("f", lr32 / q))[0]
