"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the
same seeded inputs, element by element, within |err| <= 2e-3 * (1 + |ref|)."""
import math

import numpy as np
import pytest
import torch

from mqa_workloads import WORKLOADS, make_custom, make_inputs, poison_padding
from oracle import ref
from paper_2211_05102_b200 import binding

from gpu_util import assert_close, check, plans_for, run_gpu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["tiny", "palm8b", "palm62b", "palm540b", "ragged32k"])
def test_named_configs_full_size(name):
    """The five configurations of the metric, at full size, under the heuristic's plan
    (the launch configuration the benchmark times)."""
    w = WORKLOADS[name]
    q, k, v, lengths = make_inputs(w)
    got = run_gpu(q, k, v, lengths, w.scale)
    expect = ref.mqa_decode_ref(q, k, v, lengths, w.scale)
    worst = assert_close(got, expect, name)
    print(f"{name}: max err/tol = {worst:.4f}")


@pytest.mark.parametrize("name", ["tiny", "palm8b", "palm62b"])
def test_named_configs_every_path(name):
    w = WORKLOADS[name]
    q, k, v, lengths = make_inputs(w)
    expect = ref.mqa_decode_ref(q, k, v, lengths, w.scale)
    for plan in plans_for(w.B, w.H, w.D, w.Lmax, ctas=(None, 1, 7)):
        got = run_gpu(q, k, v, lengths, w.scale, plan=plan)
        assert_close(got, expect, f"{name} {plan}")


EDGE_LENGTHS = [0, 1, 2, 3, 5, 17, 63, 64, 65, 127, 128, 129, 255, 256, 257, 300]


@pytest.mark.parametrize("D", [64, 128, 256])
@pytest.mark.parametrize("H", [1, 4, 16, 32, 48, 64])
def test_edge_lengths(H, D):
    B, Lmax = len(EDGE_LENGTHS), 300
    q, k, v, lengths = make_custom(B, H, D, Lmax, seed=1000 + H * 7 + D, lengths=EDGE_LENGTHS)
    k, v = poison_padding(k, v, lengths, 0x7FC0)     # NaN beyond every length
    expect = ref.mqa_decode_ref(q, k, v, lengths, 1.0 / math.sqrt(D))
    for plan in plans_for(B, H, D, Lmax, ctas=(None, 1, 2, 3, 7, binding.MQA_MAX_CTAS)):
        got = run_gpu(q, k, v, lengths, 1.0 / math.sqrt(D), plan=plan)
        assert_close(got, expect, f"H={H} D={D} {plan}")
        assert bool((got[0] == 0).all()), "length 0 must give an exactly zero row"


@pytest.mark.parametrize("pattern", [0x7FC0, 0x7F80, 0xFF80])
def test_padding_bits_never_reach_the_output(pattern):
    B, H, D, Lmax = 6, 48, 256, 700
    q, k, v, lengths = make_custom(B, H, D, Lmax, seed=77, lengths=[700, 1, 129, 500, 64, 333])
    expect = ref.mqa_decode_ref(q, k, v, lengths, 1 / 16)
    k2, v2 = poison_padding(k, v, lengths, pattern)
    for plan in plans_for(B, H, D, Lmax, ctas=(None, 5)):
        assert_close(run_gpu(q, k2, v2, lengths, 1 / 16, plan=plan), expect, f"{plan}")


def test_long_sequences_split_across_many_blocks():
    B, H, D, Lmax = 3, 48, 256, 20000
    q, k, v, lengths = make_custom(B, H, D, Lmax, seed=78, lengths=[20000, 7, 12345])
    expect = ref.mqa_decode_ref(q, k, v, lengths, 1 / 16)
    for plan in plans_for(B, H, D, Lmax, ctas=(None, 1, 2, 3, 7, 148, binding.MQA_MAX_CTAS)):
        assert_close(run_gpu(q, k, v, lengths, 1 / 16, plan=plan), expect, f"{plan}")


def test_short_sequences_with_large_values():
    """Lengths 2 and 3 with V scaled by 4: the case where a low-precision probability
    would show (the output is a blend of very few large rows)."""
    B, H, D, Lmax = 8, 48, 256, 8
    q, k, v, _ = make_custom(B, H, D, Lmax, seed=79)
    v = (v.float() * 4).to(torch.bfloat16)
    lengths = torch.tensor([2, 3, 2, 3, 5, 2, 3, 8], dtype=torch.int32)
    expect = ref.mqa_decode_ref(q, k, v, lengths, 1 / 16)
    for plan in plans_for(B, H, D, Lmax):
        assert_close(run_gpu(q, k, v, lengths, 1 / 16, plan=plan), expect, f"{plan}")


def test_all_equal_logits_give_the_mean():
    B, H, D, Lmax = 2, 16, 128, 400
    q, k, v, lengths = make_custom(B, H, D, Lmax, seed=80, lengths=[400, 131])
    q = torch.zeros_like(q)
    expect = ref.mqa_decode_ref(q, k, v, lengths, 0.5)
    for plan in plans_for(B, H, D, Lmax, ctas=(None, 3)):
        assert_close(run_gpu(q, k, v, lengths, 0.5, plan=plan), expect, f"{plan}")


@pytest.mark.parametrize("where", ["first", "middle", "last"])
def test_one_dominant_logit(where):
    B, H, D, Lmax = 2, 32, 256, 1000
    q, k, v, lengths = make_custom(B, H, D, Lmax, seed=81, lengths=[1000, 777])
    for b in range(B):
        n = int(lengths[b])
        j = {"first": 0, "middle": n // 2, "last": n - 1}[where]
        qm = q[b].float().mean(0)
        k[b, j] = (qm * (400.0 / float(qm @ qm))).to(torch.bfloat16)
    expect = ref.mqa_decode_ref(q, k, v, lengths, 1 / 16)
    for plan in plans_for(B, H, D, Lmax, ctas=(None, 1, 4)):
        assert_close(run_gpu(q, k, v, lengths, 1 / 16, plan=plan), expect, f"{where} {plan}")


def test_logits_that_keep_growing_along_the_sequence():
    """The running maximum rises in every tile, so the accumulator is rescaled every time."""
    B, H, D, Lmax = 2, 48, 256, 1500
    q, k, v, lengths = make_custom(B, H, D, Lmax, seed=82, lengths=[1500, 901])
    qm = q.float().mean(1)                                   # [B,D]
    ramp = torch.arange(Lmax, dtype=torch.float32) / Lmax    # 0..1
    for b in range(B):
        k[b] = (k[b].float() * 0.05 + ramp[:, None] * qm[b][None, :] * (600.0 / float(qm[b] @ qm[b]))).to(torch.bfloat16)
    expect = ref.mqa_decode_ref(q, k, v, lengths, 1 / 16)
    for plan in plans_for(B, H, D, Lmax, ctas=(None, 1, 5)):
        assert_close(run_gpu(q, k, v, lengths, 1 / 16, plan=plan), expect, f"{plan}")


def test_same_plan_is_bit_identical_and_workspace_is_reusable():
    w = WORKLOADS["palm8b"]
    q, k, v, lengths = make_inputs(w)
    ws = binding.alloc_workspace(w.B, w.H, w.D, w.Lmax)
    a = run_gpu(q, k, v, lengths, w.scale, workspace=ws)
    b = run_gpu(q, k, v, lengths, w.scale, workspace=ws)
    assert torch.equal(a, b)
    # a different problem through the same (larger) workspace, then the first again
    q2, k2, v2, l2 = make_custom(3, w.H, w.D, 500, seed=83, lengths=[500, 0, 250])
    ws_big = binding.alloc_workspace(w.B, w.H, w.D, w.Lmax)
    expect2 = ref.mqa_decode_ref(q2, k2, v2, l2, w.scale)
    run_gpu(q, k, v, lengths, w.scale, workspace=ws_big)
    assert_close(run_gpu(q2, k2, v2, l2, w.scale, workspace=ws_big), expect2, "reuse")


def test_host_entry_point_matches():
    w = WORKLOADS["palm8b"]
    q, k, v, lengths = make_inputs(w)
    out = torch.empty((w.B, w.H, w.D), dtype=torch.float32).pin_memory()
    scratch = torch.empty(binding.mqa_decode_host_scratch_bytes(w.B, w.H, w.D, w.Lmax), dtype=torch.uint8, device="cuda:0")
    binding.mqa_decode_host(q.pin_memory(), k.pin_memory(), v.pin_memory(), lengths.pin_memory(), out, w.scale, scratch)
    assert_close(out, ref.mqa_decode_ref(q, k, v, lengths, w.scale), "host entry")


def test_launch_count_is_reported():
    w = WORKLOADS["tiny"]
    q, k, v, lengths = make_inputs(w)
    run_gpu(q, k, v, lengths, w.scale)
    assert binding.mqa_last_launch_count() >= 1


@pytest.mark.parametrize("B,H,L", [(160, 16, 256), (50, 48, 512), (296, 8, 130), (64, 32, 1024)])
def test_uniform_batches_under_the_adaptive_plan(B, H, L):
    """Batches of equal tile count, where the library's own plan may share the tiles among fewer blocks than
    it launches: same results as the pinned block count, and the block count the kernel reports is the
    heuristic's."""
    D, Lmax = 256, L + 40
    lengths = [L - (i % 3) for i in range(B)]        # equal tile counts, unequal lengths
    q, k, v, ln = make_custom(B, H, D, Lmax, seed=4242 + B, lengths=lengths)
    k, v = poison_padding(k, v, ln, 0x7FC0)
    expect = ref.mqa_decode_ref(q, k, v, ln, 1.0 / math.sqrt(D))
    plan = binding.mqa_decode_plan(B, H, D, Lmax, binding.MQA_PATH_TC)
    assert plan.adaptive == 1
    ws = binding.alloc_workspace(B, H, D, Lmax)
    got = run_gpu(q, k, v, ln, 1.0 / math.sqrt(D), plan=plan, workspace=ws)
    assert_close(got, expect, f"adaptive B={B}")
    nt = (L + 127) // 128
    assert int(ws[:16].view(torch.int32)[3]) == binding.mqa_uniform_ctas(B, nt, plan.num_ctas)
    pinned = binding.Plan(plan.path, plan.num_ctas, plan.tile_rows)
    got2 = run_gpu(q, k, v, ln, 1.0 / math.sqrt(D), plan=pinned, workspace=ws)
    assert_close(got2, expect, f"pinned B={B}")
    assert int(ws[:16].view(torch.int32)[3]) == plan.num_ctas


def test_cuda_graph_capture_and_replay():
    """A decode step (cooperative launch, in-kernel merge with self-resetting arrival counters) captured in a
    CUDA graph and replayed: every replay reproduces the eager result bit for bit, on fresh inputs too."""
    B, H, D, Lmax = 24, 48, 256, 3000
    lengths = [3000 - 97 * i for i in range(B)]
    dev = torch.device("cuda:0")
    q, k, v, ln = make_custom(B, H, D, Lmax, seed=606, lengths=lengths)
    qd, kd, vd, ld = q.to(dev), k.to(dev), v.to(dev), ln.to(dev)
    out = torch.empty((B, H, D), dtype=torch.float32, device=dev)
    ws = binding.alloc_workspace(B, H, D, Lmax)
    binding.mqa_decode(qd, kd, vd, ld, out, 1 / 16, ws)            # warm-up outside the capture
    torch.cuda.synchronize()
    eager = out.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.mqa_decode(qd, kd, vd, ld, out, 1 / 16, ws)
    for _ in range(3):
        out.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, eager)
    # new queries in the captured buffers
    q2, _, _, _ = make_custom(B, H, D, Lmax, seed=607, lengths=lengths)
    qd.copy_(q2.to(dev))
    graph.replay()
    torch.cuda.synchronize()
    assert binding.mqa_check_status(ws) == binding.MQA_OK
    expect = ref.mqa_decode_ref(q2, k, v, ln, 1 / 16)
    assert_close(out.cpu(), expect, "graph replay with new q")


def test_random_shapes_and_block_counts():
    """Seeded sweep over shapes, length mixes and block counts (pinned and adaptive): every case against the
    oracle.  Exercises cut sequences with 2..40 parts, blocks without tiles, empty sequences, one-row
    sequences and uniform batches in one run."""
    rng = np.random.default_rng(20221105)
    worst = 0.0
    for case in range(36):
        D = int(rng.choice([128, 256]))
        H = int(rng.choice([1, 3, 8, 16, 17, 32, 40, 48, 64]))
        B = int(rng.integers(1, 41))
        Lmax = int(rng.choice([130, 700, 2100, 5200]))
        kind = case % 4
        if kind == 0:
            lengths = [int(x) for x in rng.integers(0, Lmax + 1, size=B)]
        elif kind == 1:
            lengths = [Lmax - int(x) for x in rng.integers(0, 100, size=B)]          # equal tile counts, mostly
        elif kind == 2:
            lengths = [int(rng.choice([0, 1, 127, 128, 129, Lmax])) for _ in range(B)]
        else:
            lengths = [Lmax] * B
        q, k, v, ln = make_custom(B, H, D, Lmax, seed=3000 + case, lengths=lengths)
        k, v = poison_padding(k, v, ln, 0x7FC0)
        scale = 1.0 / math.sqrt(D)
        expect = ref.mqa_decode_ref(q, k, v, ln, scale)
        base = binding.mqa_decode_plan(B, H, D, Lmax, binding.MQA_PATH_TC)
        pinned = binding.Plan(base.path, int(rng.integers(1, 149)), base.tile_rows)
        for plan in (base, pinned):
            got = run_gpu(q, k, v, ln, scale, plan=plan)
            worst = max(worst, assert_close(got, expect, f"case {case}: B={B} H={H} D={D} Lmax={Lmax} kind={kind} {plan}"))
    print(f"random sweep: max err/tol = {worst:.3f}")


@pytest.mark.parametrize("pin", [None, 148, 37])
def test_repeated_launches_are_bit_identical(pin):
    """Many back-to-back steps on a batch whose sequences are cut into 2..40 parts (publisher, arrival counters
    that wrap back to zero, sliced merge): every step must reproduce the first one bit for bit, and the first
    one must match the oracle.  A merge that read a part too early, or a counter that did not return to zero,
    shows up here."""
    B, H, D, Lmax = 12, 48, 256, 5200
    lengths = [5200, 130, 0, 4100, 2600, 1, 900, 5199, 3333, 128, 777, 2048]
    dev = torch.device("cuda:0")
    q, k, v, ln = make_custom(B, H, D, Lmax, seed=911, lengths=lengths)
    qd, kd, vd, ld = q.to(dev), k.to(dev), v.to(dev), ln.to(dev)
    out = torch.empty((B, H, D), dtype=torch.float32, device=dev)
    ws = binding.alloc_workspace(B, H, D, Lmax)
    plan = binding.mqa_decode_plan(B, H, D, Lmax, binding.MQA_PATH_TC)
    if pin is not None:
        plan = binding.Plan(plan.path, pin, plan.tile_rows)
    binding.mqa_decode(qd, kd, vd, ld, out, 1 / 16, ws, plan=plan)
    torch.cuda.synchronize()
    first = out.clone()
    assert_close(first.cpu(), ref.mqa_decode_ref(q, k, v, ln, 1 / 16), f"first step, pin={pin}")
    for it in range(400):
        if it % 50 == 0:
            out.fill_(float("nan"))
        binding.mqa_decode(qd, kd, vd, ld, out, 1 / 16, ws, plan=plan)
        if it % 50 == 49:
            torch.cuda.synchronize()
            assert torch.equal(out, first), f"step {it} differs"
    assert binding.mqa_check_status(ws) == binding.MQA_OK
    # the arrival counters are back at zero
    off = 256 + (B * 8 + 255) // 256 * 256
    assert int(ws[off:off + 4 * B].view(torch.int32).abs().sum()) == 0


@pytest.mark.parametrize("B,H,L", [(64, 32, 2048), (70, 48, 512), (37, 64, 1024), (74, 16, 300), (64, 48, 4096)])
def test_pair_mode_merges_halves_through_cluster_shared_memory(B, H, L):
    """Uniform batches that the heuristic runs on exactly two blocks per sequence: the launch uses clusters of
    two and the halves are merged through distributed shared memory (workspace header word 4 says so).
    Unequal lengths inside the same tile count, padding poisoned with NaN."""
    D, Lmax = 256, L
    lengths = [L - (i % 5) for i in range(B)]
    q, k, v, ln = make_custom(B, H, D, Lmax, seed=5150 + B, lengths=lengths)
    k, v = poison_padding(k, v, ln, 0x7FC0)
    expect = ref.mqa_decode_ref(q, k, v, ln, 1.0 / math.sqrt(D))
    ws = binding.alloc_workspace(B, H, D, Lmax)
    got = run_gpu(q, k, v, ln, 1.0 / math.sqrt(D), workspace=ws)
    assert_close(got, expect, f"pair mode B={B} H={H} L={L}")
    hdr = ws[:32].view(torch.int32)
    plan = binding.mqa_decode_plan(B, H, D, Lmax, binding.MQA_PATH_TC)
    import os
    clusters_on = os.environ.get("MQA_NO_CLUSTER") is None
    if clusters_on and binding.mqa_uniform_ctas(B, (L + 127) // 128, plan.num_ctas) == 2 * B and plan.num_ctas % 2 == 0:
        assert int(hdr[4]) == 1, "expected the pair path"
        assert int(hdr[3]) == 2 * B
    again = run_gpu(q, k, v, ln, 1.0 / math.sqrt(D), workspace=ws)
    assert torch.equal(got, again)
    # a ragged batch of the same shape falls back to the global-memory merge in the same cluster launch
    lengths2 = [max(1, L - 137 * i) for i in range(B)]
    q2, k2, v2, ln2 = make_custom(B, H, D, Lmax, seed=5151 + B, lengths=lengths2)
    assert_close(run_gpu(q2, k2, v2, ln2, 1.0 / math.sqrt(D), workspace=ws),
                 ref.mqa_decode_ref(q2, k2, v2, ln2, 1.0 / math.sqrt(D)), "ragged under a cluster launch")
    assert int(ws[:32].view(torch.int32)[4]) == 0


def test_cuda_graph_replay_in_pair_mode():
    """The cluster launch of pair mode inside a CUDA graph: replays reproduce the eager result bit for bit."""
    B, H, D, Lmax = 70, 16, 256, 512
    dev = torch.device("cuda:0")
    q, k, v, ln = make_custom(B, H, D, Lmax, seed=808, lengths=[512 - (i % 7) for i in range(B)])
    qd, kd, vd, ld = q.to(dev), k.to(dev), v.to(dev), ln.to(dev)
    out = torch.empty((B, H, D), dtype=torch.float32, device=dev)
    ws = binding.alloc_workspace(B, H, D, Lmax)
    binding.mqa_decode(qd, kd, vd, ld, out, 1 / 16, ws)
    torch.cuda.synchronize()
    eager = out.clone()
    assert_close(eager.cpu(), ref.mqa_decode_ref(q, k, v, ln, 1 / 16), "eager")
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.mqa_decode(qd, kd, vd, ld, out, 1 / 16, ws)
    for _ in range(3):
        out.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, eager)
    assert binding.mqa_check_status(ws) == binding.MQA_OK


def test_two_streams_with_separate_workspaces():
    """Steps enqueued alternately on two streams (separate workspaces): the cooperative launches, whose blocks
    wait for one another, must not starve each other, and both results match the oracle."""
    dev = torch.device("cuda:0")
    B, H, D, Lmax = 40, 48, 256, 3000
    qa, ka, va, la = make_custom(B, H, D, Lmax, seed=11, lengths=[3000 - 50 * i for i in range(B)])
    qb, kb, vb, lb = make_custom(B, H, D, Lmax, seed=12, lengths=[1000 + 50 * i for i in range(B)])
    ea = ref.mqa_decode_ref(qa, ka, va, la, 1 / 16)
    eb = ref.mqa_decode_ref(qb, kb, vb, lb, 1 / 16)
    a = [t.to(dev) for t in (qa, ka, va, la)]
    b = [t.to(dev) for t in (qb, kb, vb, lb)]
    oa = torch.empty((B, H, D), dtype=torch.float32, device=dev)
    ob = torch.empty_like(oa)
    wa, wb = binding.alloc_workspace(B, H, D, Lmax), binding.alloc_workspace(B, H, D, Lmax)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(30):
        binding.mqa_decode(*a, oa, 1 / 16, wa, stream=s1)
        binding.mqa_decode(*b, ob, 1 / 16, wb, stream=s2)
    torch.cuda.synchronize()
    assert binding.mqa_check_status(wa) == binding.MQA_OK and binding.mqa_check_status(wb) == binding.MQA_OK
    assert_close(oa.cpu(), ea, "stream 1")
    assert_close(ob.cpu(), eb, "stream 2")
