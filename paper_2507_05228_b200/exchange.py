"""Stage B of the single-layer pipeline on several GPUs: partial rows travel to the party that combines them.

The paper's layer has two communication stages (appendix "Communication Analysis"): (A) the CompNodes hand sharded
q, k, v rows to the AttnNodes, (B) every AttnNode_{jk} sends the rows of its (u, m, e) to the CompNode that owns
them, which then runs the post-pass (Single Layer Forward Pass algorithm: "CompNode_i gets m, e, u").  Here one rank
per GPU plays both roles:

* rank g keeps the k, v rows of the KV shards {k : k mod P = g} resident and never moves them (an AttnNode's shard;
  the token-sharded cache of the "Caching" paragraph), and owns the output rows of the query shards {j : j mod P = g};
* it computes the partials of its KV shards against every query row through ``cascade_shard_plan_resident`` +
  ``cascade_attn_partials`` (q is taken as replicated: stage A restricted to q);
* stage B is one all-to-all: the rows of query shard j go to rank j mod P.  What arrives lies in local memory before
  any kernel reads it; ``cascade_merge`` (the post-pass combine) then runs on local data only.

The routing is plain index arithmetic on the plan's Q_OFF array and is the same on CPU tensors (gloo) and GPU tensors
(NCCL); ``pack`` / ``unpack`` are separate from the collective so that the ranks can also be played one after another
in a single process.  Bytes on the wire are counted from the tensors sent and compared with the paper's closed form
beta (d + 2) H N elements per sequence.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch
import torch.distributed as dist


def owned_shards(n_shards: int, rank: int, world: int) -> np.ndarray:
    """Shard ids a rank owns: k with k mod world == rank."""
    return np.arange(rank, n_shards, world, dtype=np.int64)


def resident_kv(kv_shard_of: np.ndarray, n_kv_shards: int, rank: int, world: int):
    """The K/V rows a rank keeps: (tokens, local_shard_of, n_local).

    tokens          ascending original token ids of the rows of the rank's KV shards (also their positions: kv_pos)
    local_shard_of  for each of those rows the rank-local shard id k // world of its shard k
    n_local         number of KV shards the rank owns
    """
    kv_shard_of = np.asarray(kv_shard_of)
    assert kv_shard_of.ndim == 1, "one map for the batch"
    mine = (kv_shard_of % world) == rank
    tokens = np.flatnonzero(mine).astype(np.int32)
    local = (kv_shard_of[tokens] // world).astype(np.int32)
    return tokens, local, len(owned_shards(n_kv_shards, rank, world))


def stage_b_elements(batch: int, n_kv_shards: int, n_q: int, n_heads: int, head_dim: int) -> int:
    """Closed form of the stage-B payload in elements: beta (d + 2) H N per sequence (u has d, m and e one each)."""
    return batch * n_kv_shards * (head_dim + 2) * n_heads * n_q


def stage_b_bytes(batch: int, n_kv_shards: int, n_q: int, n_heads: int, head_dim: int, u_elt_bytes: int) -> int:
    """The same payload in bytes with u in the I/O type and m, e in fp32."""
    return batch * n_kv_shards * n_q * n_heads * (head_dim * u_elt_bytes + 8)


def stage_a_elements(batch: int, beta: int, n_tokens: int, n_heads: int, n_kv_heads: int, head_dim: int) -> int:
    """Closed form of the stage-A payload (sharded q, k, v rows to the AttnNodes): beta d (H + 2 H_KV) N elements."""
    return batch * beta * head_dim * (n_heads + 2 * n_kv_heads) * n_tokens


def layer_comm_bytes(beta: int, elt_bytes: int, head_dim: int, n_heads: int, n_kv_heads: int, n_tokens: int) -> int:
    """Both stages of one layer: CommBytes = beta F (2 d H + 2 d H_KV + 2 H) N (Section 7.1, "Communication")."""
    return elt_bytes * (stage_a_elements(1, beta, n_tokens, n_heads, n_kv_heads, head_dim) +
                        stage_b_elements(1, beta, n_tokens, n_heads, head_dim))


class StageB:
    """Routing tables of the stage-B all-to-all for one rank.

    q_off        the plan's Q_OFF array [n_q_shards + 1] (shard-major slot ranges of the query shards)
    n_kv_shards  KV shards of the whole problem (over all ranks)
    """

    def __init__(self, q_off: Sequence[int], n_kv_shards: int, rank: int, world: int):
        q_off = np.asarray(q_off, dtype=np.int64).reshape(-1)
        self.rank, self.world, self.n_kv_shards = rank, world, n_kv_shards
        self.n_q_shards = q_off.size - 1
        self.n_q = int(q_off[-1])
        # slots (shard-major row positions) owned by each rank: the ranges of its query shards, in shard order
        self.slots_of: List[np.ndarray] = []
        for h in range(world):
            ranges = [np.arange(q_off[j], q_off[j + 1]) for j in owned_shards(self.n_q_shards, h, world)]
            self.slots_of.append(np.concatenate(ranges) if ranges else np.zeros(0, dtype=np.int64))
        self.n_local_of = [len(owned_shards(n_kv_shards, s, world)) for s in range(world)]
        self.my_slots = self.slots_of[rank]

    # ---- what this rank sends
    def pack(self, o_part: torch.Tensor, m_part: torch.Tensor, l_part: torch.Tensor):
        """o_part [B, n_local, n_q, H, d], m_part / l_part [B, n_local, n_q, H] of THIS rank's KV shards.
        Returns (payload_u, payload_stats, split_u, split_stats): flat send buffers ordered by destination rank and
        the number of elements for each destination."""
        B, n_local, n_q, H, d = o_part.shape
        assert n_local == self.n_local_of[self.rank] and n_q == self.n_q
        stats = torch.stack((m_part, l_part), dim=-1)  # [B, n_local, n_q, H, 2]
        us, ss, split_u, split_s = [], [], [], []
        for h in range(self.world):
            idx = torch.from_numpy(self.slots_of[h]).to(o_part.device)
            us.append(o_part.index_select(2, idx).reshape(-1))
            ss.append(stats.index_select(2, idx).reshape(-1))
            split_u.append(us[-1].numel())
            split_s.append(ss[-1].numel())
        return torch.cat(us), torch.cat(ss), split_u, split_s

    # ---- what this rank receives
    def recv_splits(self, B: int, H: int, d: int):
        rows = self.my_slots.size
        return ([B * self.n_local_of[s] * rows * H * d for s in range(self.world)],
                [B * self.n_local_of[s] * rows * H * 2 for s in range(self.world)])

    def unpack(self, recv_u: torch.Tensor, recv_stats: torch.Tensor, B: int, H: int, d: int):
        """Flat receive buffers (ordered by source rank) -> (u [B, n_kv_shards, rows, H, d], m, l [B, n_kv_shards,
        rows, H]) for the rows this rank owns, parts in global KV-shard order, rows in shard-major order."""
        rows = self.my_slots.size
        u = recv_u.new_empty((B, self.n_kv_shards, rows, H, d))
        st = recv_stats.new_empty((B, self.n_kv_shards, rows, H, 2))
        split_u, split_s = self.recv_splits(B, H, d)
        ou = os_ = 0
        for s in range(self.world):
            n_loc = self.n_local_of[s]
            # source s holds the KV shards s, s + world, s + 2 world, ...
            u[:, s::self.world] = recv_u[ou:ou + split_u[s]].view(B, n_loc, rows, H, d)
            st[:, s::self.world] = recv_stats[os_:os_ + split_s[s]].view(B, n_loc, rows, H, 2)
            ou += split_u[s]
            os_ += split_s[s]
        return u, st[..., 0].contiguous(), st[..., 1].contiguous()

    def exchange(self, o_part: torch.Tensor, m_part: torch.Tensor, l_part: torch.Tensor, group=None):
        """pack -> all-to-all -> unpack.  Returns (u, m, l, bytes_sent); bytes_sent counts every payload byte this
        rank hands to the collective, its own rows included (the paper counts every AttnNode -> CompNode transfer)."""
        B, _, _, H, d = o_part.shape
        send_u, send_s, in_u, in_s = self.pack(o_part, m_part, l_part)
        out_u, out_s = self.recv_splits(B, H, d)
        recv_u = send_u.new_empty(sum(out_u))
        recv_s = send_s.new_empty(sum(out_s))
        if self.world == 1:
            recv_u.copy_(send_u)
            recv_s.copy_(send_s)
        else:
            dist.all_to_all_single(recv_u, send_u, out_u, in_u, group=group)
            dist.all_to_all_single(recv_s, send_s, out_s, in_s, group=group)
        nbytes = send_u.numel() * send_u.element_size() + send_s.numel() * send_s.element_size()
        return (*self.unpack(recv_u, recv_s, B, H, d), nbytes)


def deliver_in_process(stages: List[StageB], packed: List[Tuple[torch.Tensor, torch.Tensor, list, list]], B: int, H: int,
                       d: int):
    """The all-to-all played inside one process: packed[s] is rank s's ``pack`` result; returns each rank's
    ``unpack`` result.  Lets one GPU (or one CPU process) run every rank of the exchange in turn."""
    world = len(stages)
    out = []
    for g in range(world):
        us, ss = [], []
        for s in range(world):
            send_u, send_s, in_u, in_s = packed[s]
            ou, os_ = sum(in_u[:g]), sum(in_s[:g])
            us.append(send_u[ou:ou + in_u[g]])
            ss.append(send_s[os_:os_ + in_s[g]])
        out.append(stages[g].unpack(torch.cat(us), torch.cat(ss), B, H, d))
    return out


class RankAttention:
    """One rank's share of a layer's attention: resident K/V, partials, stage-B exchange, local post-pass.

    q_shard_of / kv_shard_of are the maps of the WHOLE sequence (one map for the batch); k_res / v_res passed to
    ``run`` hold only this rank's resident rows ``self.tokens`` in that order.
    """

    def __init__(self, q_shard_of: np.ndarray, kv_shard_of: np.ndarray, n_q_shards: int, n_kv_shards: int, rank: int,
                 world: int, q_pos_offset: int = 0, causal: bool = True):
        from . import binding as cb
        if world > n_kv_shards:
            raise ValueError("more ranks than KV shards: some rank would hold no K/V rows")
        self.cb = cb
        self.rank, self.world = rank, world
        self.tokens, local_map, self.n_local = resident_kv(kv_shard_of, n_kv_shards, rank, world)
        self.plan = cb.cascade_shard_plan_resident(q_shard_of, local_map, self.tokens, n_q_shards, self.n_local,
                                                   q_pos_offset, causal)
        self.stage = StageB(self.plan.get("q_off")[0].reshape(-1), n_kv_shards, rank, world)
        q_idx = self.plan.get("q_idx")[0].reshape(-1)
        self.owned_tokens = q_idx[self.stage.my_slots]  # output row r of ``run`` is this token
        self.parts = None
        self._gather = None

    def partials(self, q: torch.Tensor, k_res: torch.Tensor, v_res: torch.Tensor, scale: float, workspace=None):
        self.parts = self.cb.cascade_attn_partials(self.plan, q, k_res, v_res, scale, out=self.parts,
                                                   workspace=workspace)
        return self.parts

    def combine(self, u: torch.Tensor, m: torch.Tensor, l: torch.Tensor, want_lse: bool = True):
        """Post-pass over what arrived: rows in the order of ``owned_tokens``.  A rank that owns no query shard (more
        ranks than query shards, e.g. a decode step with one query row) has nothing to combine."""
        if u.shape[2] == 0:
            B, _, _, H, d = u.shape
            return u.new_empty((B, 0, H, d)), (m.new_empty((B, 0, H)) if want_lse else None)
        return self.cb.cascade_merge(u, m, l, 0, want_lse=want_lse)

    def combine_in_place(self, sources, want_lse: bool = True):
        """Stage B and the post-pass in one kernel (``cascade_merge_peers``): ``sources[s]`` are the partial buffers
        (o_part, m_part, l_part) of rank s, left where rank s wrote them and reachable from this GPU - the rank's own
        tensors, or a peer's buffers mapped into this process.  No packing, no all-to-all, no staging copy: the kernel
        gathers this rank's rows from every source with plain loads.  Rows in the order of ``owned_tokens``."""
        if self.stage.my_slots.size == 0:
            B, _, _, H, d = sources[0][0].shape
            return sources[0][0].new_empty((B, 0, H, d)), None
        if self._gather is None:
            self._gather = torch.from_numpy(self.stage.my_slots.astype(np.int32)).to(sources[0][0].device)
        return self.cb.cascade_merge_peers(sources, self._gather, self.stage.my_slots.size, want_lse=want_lse)

    def run(self, q, k_res, v_res, scale, group=None, workspace=None):
        """partials -> stage-B all-to-all -> post-pass.  Returns (o [B, owned rows, H, d], lse, bytes_sent)."""
        parts = self.partials(q, k_res, v_res, scale, workspace=workspace)
        u, m, l, nbytes = self.stage.exchange(*parts, group=group)
        o, lse = self.combine(u, m, l)
        return o, lse, nbytes

    def destroy(self):
        self.plan.destroy()
