"""Expert-parallel plumbing on CPU: two gloo ranks run `ExpertParallelMoE.forward` with its real
all-to-all exchanges; the oracle's stage functions stand in for the GPU stages.  The ranks' outputs
must equal the oracle's single-process layer on the whole batch, bit for bit.  Also the in-process driver
(`run_local`) and the planning helpers."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


class OracleStages:
    """The three stages of the expert-parallel layer computed by the oracle on CPU tensors."""

    def __init__(self, w13c, w13s, w2c, w2s, E):
        self.w13c, self.w13s, self.w2c, self.w2s, self.E = w13c, w13s, w2c, w2s, E   # LOCAL experts

    def dispatch(self, x, ids, wts):
        import oracle
        xb, idn, wn = x.numpy().view(np.uint16), ids.numpy(), wts.numpy()
        k = idn.shape[1]
        offsets, sorted_pair, pos = oracle.permute(idn, self.E)
        codes, scales = oracle.quantize_act(xb)
        tok = sorted_pair // k
        return dict(codes=torch.from_numpy(codes[tok]), scales=torch.from_numpy(scales[tok]),
                    weights=torch.from_numpy(wn.reshape(-1)[sorted_pair].copy()),
                    offsets=torch.from_numpy(offsets.astype(np.int32)),
                    pos_of_pair=torch.from_numpy(pos.astype(np.int32)))

    contrib_dtype = torch.float32

    def experts(self, codes, scales, weights, offsets, out):
        """-> fp32 rows of the down projection (the oracle's combine applies the pair weight itself)."""
        import oracle
        c, s, off = codes.numpy(), scales.numpy(), offsets.numpy()
        H = c.shape[1]
        y = np.zeros((c.shape[0], H), dtype=np.float32)
        for e in range(len(off) - 1):
            a, b = off[e], off[e + 1]
            if a == b:
                continue
            _, gu = oracle.linear_q(c[a:b], s[a:b], self.w13c[e], self.w13s[e])
            hc, hs = oracle.quantize_act(oracle.swiglu(gu))
            y[a:b], _ = oracle.linear_q(hc, hs, self.w2c[e], self.w2s[e])
        out.copy_(torch.from_numpy(y))
        return out

    def combine(self, contrib_sorted, ids, pos_of_pair):
        import oracle
        by_pair = contrib_sorted.numpy()[pos_of_pair.numpy()]
        # the weights travelled with the rows only for the GPU stages; the oracle's combine takes them here
        return torch.from_numpy(oracle.combine(by_pair, ids.numpy(), self._wts).view(np.int16))


def _case():
    from paper_2604_07853_b200 import inputs
    import oracle
    c = inputs.moe_case(21, 50, h=256, i=128, e=8, k=2, zipf_s=1.1)
    w13c, w13s = oracle.quantize_weight(c.w13)
    w2c, w2s = oracle.quantize_weight(c.w2)
    return c, (w13c, w13s, w2c, w2s)


def _rank_inputs(c, lo, hi):
    return (torch.from_numpy(c.x[lo:hi].view(np.int16).copy()), torch.from_numpy(c.ids[lo:hi].copy()),
            torch.from_numpy(c.weights[lo:hi].copy()))


def _make_rank(c, q, rank, world, group=None):
    from paper_2604_07853_b200.expert_parallel import ExpertParallelMoE, expert_range
    lo, hi = expert_range(rank, world, c.E)
    st = OracleStages(q[0][lo:hi], q[1][lo:hi], q[2][lo:hi], q[3][lo:hi], c.E)
    return ExpertParallelMoE(st, rank, world, c.E, group)


SPLITS = {2: [0, 31, 50], 4: [0, 0, 20, 21, 50]}     # uneven token shares, one rank without tokens


def _worker(rank: int, world: int, port: int, tmp: str):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    c, q = _case()
    ep = _make_rank(c, q, rank, world)
    lo, hi = SPLITS[world][rank], SPLITS[world][rank + 1]
    x, ids, wts = _rank_inputs(c, lo, hi)
    ep.stages._wts = wts.numpy()
    out = ep.forward(x, ids, wts)
    np.save(os.path.join(tmp, f"out{rank}.npy"), out.numpy().view(np.uint16))
    dist.barrier()
    dist.destroy_process_group()


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def test_two_gloo_ranks_equal_the_single_process_layer(tmp_path):
    import oracle
    mp.spawn(_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
    c, q = _case()
    ref = oracle.moe(c.x, c.ids, c.weights, *q)
    got = np.concatenate([np.load(tmp_path / f"out{r}.npy") for r in range(2)])
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("world", [1, 2, 4])
def test_in_process_driver_equals_the_single_process_layer(world):
    import oracle
    from paper_2604_07853_b200.expert_parallel import run_local
    c, q = _case()
    split = SPLITS.get(world, [0, 50])
    ranks = [_make_rank(c, q, r, world) for r in range(world)]
    inputs_ = [_rank_inputs(c, split[r], split[r + 1]) for r in range(world)]
    for ep, inp in zip(ranks, inputs_):
        ep.stages._wts = inp[2].numpy()
    outs = run_local(ranks, inputs_)
    got = np.concatenate([o.numpy().view(np.uint16) for o in outs])
    assert np.array_equal(got, oracle.moe(c.x, c.ids, c.weights, *q))


def test_planning_helpers():
    from paper_2604_07853_b200.expert_parallel import expert_range, group_offsets, send_counts
    assert [expert_range(r, 4, 128) for r in range(4)] == [(0, 32), (32, 64), (64, 96), (96, 128)]
    with pytest.raises(ValueError):
        expert_range(0, 3, 128)
    off = torch.tensor([0, 2, 2, 5, 9, 9, 9, 10, 12], dtype=torch.int32)
    sc = send_counts(off, 2)
    assert sc.tolist() == [[2, 0, 3, 4], [0, 0, 1, 2]] and sc.dtype == torch.int64
    assert group_offsets(sc[1], "cpu").tolist() == [0, 0, 0, 1, 3]
    assert send_counts(off, 8).reshape(-1).tolist() == [2, 0, 3, 4, 0, 0, 1, 2]
