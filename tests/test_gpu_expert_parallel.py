"""GPU parity of the expert-parallel form of the FP8 MoE layer: the dispatch stage against the oracle,
and the whole layer, run as 1, 2, 4 or 8 ranks in one process on one GPU (exchanges by slicing), bytewise
equal to the single-GPU layer (App. C: a row's result does not depend on what else is in the batch, so
it cannot depend on which GPU holds its expert either)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_07853_b200 import binding, build, inputs
from paper_2604_07853_b200.expert_parallel import CudaStages, ExpertParallelMoE, expert_range, run_local
from util import bits_to_torch, to_dev, torch_to_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = binding.Context(0)
    yield c
    assert c.poll() == 0
    c.close()


def device_case(ctx, case):
    x, ids, wts = bits_to_torch(case.x), to_dev(case.ids), to_dev(case.weights)
    w13 = ctx.quantize_weight(bits_to_torch(case.w13))
    w2 = ctx.quantize_weight(bits_to_torch(case.w2))
    return x, ids, wts, w13, w2


def test_dispatch_stage_matches_the_oracle(ctx):
    case = inputs.moe_case(31, 333, h=512, i=256, e=16, k=4, zipf_s=1.1)
    x, ids, wts, _, _ = device_case(ctx, case)
    d = ctx.moe_dispatch(x, ids, wts, case.E)
    assert ctx.poll() == 0
    off, srt, pos = oracle.permute(case.ids, case.E)
    assert np.array_equal(d["offsets"].cpu().numpy(), off)
    assert np.array_equal(d["pos_of_pair"].cpu().numpy(), pos)
    codes, scales = oracle.quantize_act(case.x)
    tok = srt // case.k
    assert np.array_equal(d["codes"].cpu().numpy(), codes[tok])
    assert np.array_equal(d["scales"].cpu().numpy().view(np.uint32), scales[tok].view(np.uint32))
    assert np.array_equal(d["weights"].cpu().numpy(), case.weights.reshape(-1)[srt])


def run_ranks(ctx, case, world, split):
    x, ids, wts, w13, w2 = device_case(ctx, case)
    ref = ctx.moe_fwd(x, ids, wts, *w13, *w2).clone()
    ranks, inp = [], []
    for r in range(world):
        lo, hi = expert_range(r, world, case.E)
        st = CudaStages(ctx, (w13[0][lo:hi], w13[1][lo:hi]), (w2[0][lo:hi], w2[1][lo:hi]), case.E)
        ranks.append(ExpertParallelMoE(st, r, world, case.E))
        a, b = split[r], split[r + 1]
        inp.append((x[a:b].contiguous(), ids[a:b].contiguous(), wts[a:b].contiguous()))
    outs = run_local(ranks, inp)
    assert ctx.poll() == 0
    assert torch.equal(torch.cat(outs), ref)
    return ref


def even_split(m, world):
    return [m * r // world for r in range(world + 1)]


def test_one_rank_three_stages_equal_the_fused_layer(ctx):
    case = inputs.moe_case(32, 200, h=256, i=128, e=8, k=2)
    ref = run_ranks(ctx, case, 1, [0, 200])
    # and the fused layer equals the oracle end to end within the layer's tolerance
    q13 = oracle.quantize_weight(case.w13)
    q2 = oracle.quantize_weight(case.w2)
    o = inputs.bf16_bits_to_f32(oracle.moe(case.x, case.ids, case.weights, *q13, *q2)).astype(np.float64)
    g = inputs.bf16_bits_to_f32(torch_to_bits(ref)).astype(np.float64)
    assert np.linalg.norm(g - o) / np.linalg.norm(o) < 5e-3


@pytest.mark.parametrize("world", [2, 4, 8])
def test_ranks_equal_the_single_gpu_layer(ctx, world):
    case = inputs.moe_case(33 + world, 600, h=512, i=256, e=16, k=4, zipf_s=1.1)
    run_ranks(ctx, case, world, even_split(600, world))


def test_uneven_token_shares_and_a_rank_without_tokens(ctx):
    case = inputs.moe_case(40, 257, h=256, i=256, e=8, k=2, zipf_s=1.1)
    run_ranks(ctx, case, 4, [0, 0, 130, 131, 257])


def test_experts_without_rows_and_ranks_without_rows(ctx):
    # 3 tokens x 2 experts out of 32: most experts, and some ranks, receive nothing
    case = inputs.moe_case(41, 3, h=256, i=128, e=32, k=2)
    run_ranks(ctx, case, 8, [0, 1, 1, 2, 2, 2, 3, 3, 3])


def test_decode_layer_shape_on_four_ranks(ctx):
    case = inputs.config3()
    run_ranks(ctx, case, 4, even_split(case.x.shape[0], 4))


def test_forward_over_a_one_rank_nccl_group(ctx):
    """The per-process driver with its real collectives (all_to_all_single on device tensors); one rank is
    all this machine has, so the exchanges are self-sends, but counts, splits and buffers take the NCCL path."""
    import socket
    import torch.distributed as dist
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda", 0))
    try:
        case = inputs.moe_case(42, 300, h=256, i=128, e=8, k=2, zipf_s=1.1)
        x, ids, wts, w13, w2 = device_case(ctx, case)
        ref = ctx.moe_fwd(x, ids, wts, *w13, *w2).clone()
        ep = ExpertParallelMoE(CudaStages(ctx, w13, w2, case.E), 0, 1, case.E)
        out = ep.forward(x, ids, wts)
        assert ctx.poll() == 0
        assert torch.equal(out, ref)
    finally:
        dist.destroy_process_group()


def test_stage_argument_checks(ctx):
    dev = torch.device("cuda", 0)
    x = torch.zeros((4, 192), dtype=torch.bfloat16, device=dev)        # H not a multiple of 128
    ids = torch.zeros((4, 1), dtype=torch.int32, device=dev)
    wts = torch.ones((4, 1), dtype=torch.float32, device=dev)
    with pytest.raises(binding.QarlError):
        ctx.moe_dispatch(x, ids, wts, 4)
    # no tokens: the offsets are all zero and nothing else is touched
    d = ctx.moe_dispatch(torch.zeros((0, 256), dtype=torch.bfloat16, device=dev),
                         torch.zeros((0, 2), dtype=torch.int32, device=dev),
                         torch.zeros((0, 2), dtype=torch.float32, device=dev), 8)
    assert ctx.poll() == 0 and d["offsets"].cpu().tolist() == [0] * 9
