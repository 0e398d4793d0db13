"""A step spread over several devices (zo_set_query_shard / zo_loss_buffer / zo_apply_update).

With one GPU the ranks are emulated one after another: each "rank" has its own context, workspace
and copy of the B tensors, runs its block of queries to completion, then the loss arrays are summed
as the all-reduce would and every rank applies the update.  No kernel waits for another.  The result
must be the whole step's: same losses, same g, same B, bit for bit (each replica's arithmetic does
not depend on which other replicas share its pass, for launches that are not split along K)."""
import numpy as np
import pytest

from workloads import ModelSpec, config, make_decoder_problem, make_linear_problem
from workloads.spec import ARCH_LLAMA, ARCH_OPT

from gpu_util import run_gpu, run_oracle, update_rel_err

pytestmark = pytest.mark.gpu


def _sharded(spec, p, seed, world, q=None, schedule=None):
    import torch
    import paper_2409_15520_b200 as zo
    q = spec.q if q is None else q
    ranks = []
    for rank in range(world):
        est = zo.Estimator(zo.make_config(spec, max_q=q))
        prob = zo.DeviceProblem(p, spec.bf16)
        if schedule:
            est.set_schedule(schedule)
        begin, count = zo.query_shard(q, world, rank)
        est.set_query_shard(begin, count)
        est.step(prob, spec.E, spec.S, seed, q, spec.eps, 0.0)
        ranks.append((est, prob, begin, count))
    torch.cuda.synchronize()
    bufs = [est.loss_buffer() for est, *_ in ranks]
    for (est, prob, begin, count), buf in zip(ranks, bufs):
        own = buf[:2 * q].cpu().numpy()
        mask = np.zeros(2 * q, bool)
        mask[2 * begin:2 * (begin + count)] = True
        assert np.all(own[~mask] == 0.0) and np.all(own[mask] != 0.0)     # own block filled, the rest zeroed
    total = torch.stack([b[:2 * q] for b in bufs]).sum(0)                 # what the all-reduce leaves everywhere
    outs = []
    for (est, prob, *_), buf in zip(ranks, bufs):
        buf[:2 * q].copy_(total)
        est.apply_update(prob, seed, q, spec.eps, spec.lr)
        losses, g = est.losses()
        outs.append(dict(losses=losses.astype(np.float64), g=g.astype(np.float64), B=prob.B_numpy()))
        est.close()
    return outs


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_linear_step_equals_the_whole_step_and_the_oracle(world):
    spec = config("linear_fp32")
    p = make_linear_problem(spec, seed=1234, b_std=0.02)
    q = 5                                                   # uneven blocks: 3+2, 2+2+1
    whole = run_gpu(spec, p, 3, q=q)
    ref = run_oracle(spec, p, p["X"], p["target"], 3, q=q)
    for out in _sharded(spec, p, 3, world, q=q):
        assert np.array_equal(out["losses"], whole["losses"])
        assert np.array_equal(out["g"], whole["g"])
        assert all(np.array_equal(a, b) for a, b in zip(out["B"], whole["B"]))
        assert np.allclose(out["losses"], ref["losses"], rtol=1e-4, atol=0)
        assert np.all(np.abs(out["g"] - ref["g"]) <= 1e-2 * np.abs(ref["g"]).max())
        assert update_rel_err(spec, p, out["B"], ref["B"]) < 1e-3


@pytest.mark.parametrize("arch,bf16,schedule", [(ARCH_LLAMA, False, None), (ARCH_OPT, True, None),
                                                (ARCH_LLAMA, True, "inner_only")])
def test_sharded_decoder_step_equals_the_whole_step(arch, bf16, schedule):
    # 384 rows per replica: no launch is small enough to be split along K, so bit-identity holds
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=bf16, n_layers=2, d_model=256, n_heads=4,
                     d_ffn=512, vocab=777, max_seq=96, lora_rank=8, E=4, S=96, q=4, n_labelled=6, eps=1e-2, lr=1e-2)
    p = make_decoder_problem(spec, seed=5, b_std=0.03)
    whole = run_gpu(spec, p, 21)
    outs = _sharded(spec, p, 21, 2, schedule=schedule)
    for out in outs:
        assert np.array_equal(out["losses"], whole["losses"]), (out["losses"], whole["losses"])
        assert np.array_equal(out["g"], whole["g"])
        assert all(np.array_equal(a, b) for a, b in zip(out["B"], whole["B"]))
    if not bf16:
        ref = run_oracle(spec, p, p["tokens"], p["labels"], 21)
        assert np.allclose(outs[0]["losses"], ref["losses"], rtol=1e-4, atol=0)
        assert update_rel_err(spec, p, outs[0]["B"], ref["B"]) < 1e-3


def test_shard_arguments_and_deferred_update_on_one_context():
    import paper_2409_15520_b200 as zo
    spec = config("linear_fp32")
    p = make_linear_problem(spec, seed=1234, b_std=0.02)
    whole = run_gpu(spec, p, 9)
    est, prob = zo.Estimator(zo.make_config(spec)), zo.DeviceProblem(p, False)
    with pytest.raises(zo.ZoError):
        est.set_query_shard(0, spec.q + 1)                  # beyond max_q
    with pytest.raises(zo.ZoError):
        est.set_query_shard(-1, 1)
    est.set_query_shard(1, 1)                               # fine for a step of q = 2 ...
    with pytest.raises(zo.ZoError):
        est.step(prob, spec.E, spec.S, 9, 1, spec.eps, spec.lr)   # ... but reaches past a step of q = 1
    with pytest.raises(zo.ZoError):
        est.set_query_shard(spec.q, 1)
    # an unsharded step with lr = 0, its update applied afterwards, is the whole step
    est.set_query_shard(0, 0)
    est.step(prob, spec.E, spec.S, 9, spec.q, spec.eps, 0.0)
    assert np.array_equal(prob.B_numpy()[0], np.asarray(p["B"], np.float32).reshape(prob.B_numpy()[0].shape))
    with pytest.raises(zo.ZoError):
        est.apply_update(prob, 9, spec.q + 1, spec.eps, spec.lr)
    est.apply_update(prob, 9, spec.q, spec.eps, spec.lr)
    losses, g = est.losses()
    assert np.array_equal(losses.astype(np.float64), whole["losses"]) and np.array_equal(g.astype(np.float64), whole["g"])
    assert np.array_equal(prob.B_numpy()[0], whole["B"][0])
    est.close()


def test_nonfinite_loss_from_another_rank_blocks_the_update():
    import paper_2409_15520_b200 as zo
    spec = config("linear_fp32")
    p = make_linear_problem(spec, seed=1234, b_std=0.02)
    est, prob = zo.Estimator(zo.make_config(spec)), zo.DeviceProblem(p, False)
    est.set_query_shard(0, 1)
    est.step(prob, spec.E, spec.S, 9, spec.q, spec.eps, 0.0)
    before = prob.B_numpy()[0].copy()
    buf = est.loss_buffer()
    buf[2:2 * spec.q] = float("inf")                        # "received" from the rank that owns query 1
    est.apply_update(prob, 9, spec.q, spec.eps, spec.lr)
    with pytest.raises(zo.ZoError) as ei:
        est.losses()
    assert ei.value.status == 6                             # ZO_ERR_NONFINITE
    assert np.array_equal(prob.B_numpy()[0], before)
    est.close()


def test_fault_on_one_rank_blocks_the_update_on_every_rank():
    """Two emulated ranks; rank 1 is given a token id outside the vocabulary.  Its status word travels
    with the losses (the fault slot at the end of the loss array), so after the sum neither rank updates
    its B: rank 1 reports its own fault, rank 0 that another device faulted."""
    import torch
    import paper_2409_15520_b200 as zo
    spec = ModelSpec(arch=ARCH_LLAMA, bf16=False, n_layers=1, d_model=64, n_heads=2, d_ffn=96, vocab=101,
                     max_seq=16, lora_rank=4, E=2, S=16, q=2, n_labelled=3, eps=1e-2, lr=1e-2)
    p = make_decoder_problem(spec, seed=5, b_std=0.03)
    ranks = []
    for rank in range(2):
        est, prob = zo.Estimator(zo.make_config(spec, max_shard_q=1)), zo.DeviceProblem(p, False)
        est.set_query_shard(rank, 1)
        tokens = prob.tokens.clone()
        if rank == 1:
            tokens[0, 3] = spec.vocab + 7
        est.step(prob, spec.E, spec.S, 21, spec.q, spec.eps, 0.0, tokens=tokens)
        ranks.append((est, prob))
    torch.cuda.synchronize()
    bufs = [est.loss_buffer() for est, _ in ranks]
    assert bufs[0].numel() == 2 * spec.q + 1
    assert bufs[0][-1].item() == 0.0 and bufs[1][-1].item() == 1.0
    total = torch.stack(bufs).sum(0)                      # the all-reduce of the whole array
    before = [prob.B_numpy() for _, prob in ranks]
    codes = []
    for (est, prob), buf in zip(ranks, bufs):
        buf.copy_(total)
        est.apply_update(prob, 21, spec.q, spec.eps, spec.lr)
        with pytest.raises(zo.ZoError) as ei:
            est.losses()
        codes.append(ei.value.status)
    assert codes == [7, 1]                                # ZO_ERR_STATE (peer fault), ZO_ERR_INVALID_ARG (own)
    for (est, prob), b0 in zip(ranks, before):
        assert all(np.array_equal(a, b) for a, b in zip(prob.B_numpy(), b0))
        est.close()


def test_shard_sized_workspace_and_reset_after_a_sharded_step():
    """max_shard_q sizes the activation workspace for the shard alone (half the replicas here); the step
    helper leaves the context unsharded, and a whole step is then refused by a context sized for shards."""
    import ctypes as C
    import paper_2409_15520_b200 as zo
    from paper_2409_15520_b200 import binding as b
    spec = ModelSpec(arch=ARCH_OPT, tie_lm_head=True, bf16=True, n_layers=2, d_model=256, n_heads=4, d_ffn=512,
                     vocab=777, max_seq=96, lora_rank=8, E=4, S=96, q=4, n_labelled=6, eps=1e-2, lr=1e-2)
    full, half = zo.make_config(spec), zo.make_config(spec, max_shard_q=2)
    nb_full, nb_half = b.zo_workspace_bytes(C.byref(full)), b.zo_workspace_bytes(C.byref(half))
    # the replicated activations (hidden, normed, q|k|v, MLP) of the 4 replicas no longer provided for
    assert nb_full - nb_half > 4 * 384 * (5 * 256 + 512) * 2
    p = make_decoder_problem(spec, seed=5, b_std=0.03)
    whole = run_gpu(spec, p, 21)
    est, prob = zo.Estimator(half), zo.DeviceProblem(p, True)
    # world size 1 with an explicit block: rank 0 of 2 runs queries 0..1, "receives" the rest from a full run
    est.set_query_shard(0, 2)
    est.step(prob, spec.E, spec.S, 21, spec.q, spec.eps, 0.0)
    est.set_query_shard(0, 0)
    buf = est.loss_buffer()
    assert np.array_equal(buf[:4].cpu().numpy().astype(np.float32).astype(np.float64), whole["losses"][:4])
    assert np.all(buf[4:].cpu().numpy() == 0.0)
    with pytest.raises(zo.ZoError) as ei:                 # 4 queries in one step do not fit this workspace
        est.step(prob, spec.E, spec.S, 21, spec.q, spec.eps, 0.0)
    assert ei.value.status == 1
    est.close()
    est2, prob2 = zo.Estimator(full), zo.DeviceProblem(p, True)
    zo.sharded_step(est2, prob2, spec.E, spec.S, 21, spec.q, spec.eps, spec.lr, rank=0, world_size=1)
    est2.step(prob2, spec.E, spec.S, 22, spec.q, spec.eps, 0.0)   # a plain step afterwards is a whole step
    l2, _ = est2.losses()
    assert np.all(l2 != 0.0)
    assert all(np.array_equal(a, b_) for a, b_ in zip(prob2.B_numpy(), whole["B"]))
    est2.close()
