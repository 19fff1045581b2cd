"""One verification level with the vocabulary sharded over ranks: the exchanges around the library's three
per-rank calls (``ShardedLevelCall.stats / decide / pick``).

The library never talks to another rank; what crosses ranks is two small all-gathers (a stats record of
about 12 bytes per logits row and a mass record of 16 bytes per sequence) and one max-reduction of the
token.  ``verify_level_vocab_parallel`` does them with ``torch.distributed`` (one process per GPU, NCCL);
``verify_level_sharded_on_one_device`` runs every rank's calls one after the other on a single GPU and
concatenates the records instead, which computes exactly the same thing and is how the path is tested
where only one GPU is at hand.  No arithmetic of the method happens here.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch


def gather_records(record: torch.Tensor, group=None) -> torch.Tensor:
    """Every rank's record, concatenated in rank order (the layout ``decide`` and ``pick`` read)."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    parts = [torch.empty_like(record) for _ in range(world)]
    dist.all_gather(parts, record, group=group)
    return torch.cat(parts).contiguous()


def verify_level_vocab_parallel(call, group=None):
    """Run one level on this rank's ``call`` (any object with stats / decide / pick as ShardedLevelCall has);
    returns (accepted_len, next_token), identical on every rank."""
    import torch.distributed as dist
    stats = gather_records(call.stats(), group)
    accepted_len, mass = call.decide(stats)
    masses = gather_records(mass, group)
    token = call.pick(masses).clone()
    dist.all_reduce(token, op=dist.ReduceOp.MAX, group=group)      # -1 everywhere but on the rank that holds the token
    return accepted_len, token


def shard_vocabulary(t: torch.Tensor, n_ranks: int) -> List[torch.Tensor]:
    """[..., V] -> n_ranks contiguous slices [..., V / n_ranks] (what a vocabulary-parallel LM head would hold)."""
    V = t.shape[-1]
    if V % n_ranks:
        raise ValueError("the vocabulary must divide evenly over the ranks")
    step = V // n_ranks
    return [t[..., r * step:(r + 1) * step].contiguous() for r in range(n_ranks)]


def verify_level_sharded_on_one_device(calls: Sequence) -> tuple:
    """All ranks' calls on one device, phase by phase, each kernel running to completion before the next
    rank's (no kernel waits for another): the records are concatenated where the ranks would all-gather."""
    stats = torch.cat([c.stats() for c in calls]).contiguous()
    decided = [c.decide(stats) for c in calls]
    masses = torch.cat([m for _, m in decided]).contiguous()
    tokens = torch.stack([c.pick(masses) for c in calls])
    return [a for a, _ in decided], tokens.max(dim=0).values


def _drive_chain(calls, gather, reduce_max):
    """The order of calls and exchanges of a sharded chain, for the ranks in ``calls`` (one in a distributed run,
    all of them when one device plays every rank)."""
    stats = gather([c.stats() for c in calls])
    for level in reversed(range(calls[0].L)):
        gathers = gather([c.gather(level) for c in calls])
        masses = gather([c.decide(level, stats, gathers) for c in calls])
        token = reduce_max([c.pick(level, masses) for c in calls])
        for c in calls:
            c.handoff(level, token)
    return calls[0].out


def verify_chain_vocab_parallel(call, group=None):
    """The whole chain on this rank's ``call`` (a ShardedChainCall); returns its outputs, identical on every rank."""
    import torch.distributed as dist

    def reduce_max(tokens):
        token = tokens[0].clone()
        dist.all_reduce(token, op=dist.ReduceOp.MAX, group=group)
        return token
    return _drive_chain([call], lambda recs: gather_records(recs[0], group), reduce_max)


def verify_chain_sharded_on_one_device(calls: Sequence):
    """All ranks' chain calls on one device, phase by phase (see verify_level_sharded_on_one_device)."""
    return _drive_chain(list(calls), lambda recs: torch.cat(list(recs)).contiguous(),
                        lambda tokens: torch.stack(list(tokens)).max(dim=0).values.contiguous())
