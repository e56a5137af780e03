"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded inputs.  Integer outputs must be bit-identical; the combine must satisfy
|gpu - oracle| <= 1e-2 + 1e-2 |oracle| against the oracle's fp32 accumulation."""
import numpy as np
import pytest
import torch

import oracle as O
import workloads as W
from gpu_util import (assert_combine_close, bf16_tensor_from_bits, bits_from_bf16_tensor, make_step,
                      oracle_assign, u32)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cb():
    import paper_2609_36959_b200 as cb
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    return cb


def check_index_stages(cb, w, step, seed):
    """stats, assign and the index half of permute, compared in full. Returns the oracle results."""
    step.stats()
    step.assign(seed)
    cb.permute_index(step.assigned_slot, w.D, step.dest_counts, step.dest_offsets, step.row_of_pair,
                     step.pair_of_row, step.workspace)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0

    coact, load = O.coact_stats(w.topk_ids, w.E)
    assert (u32(step.coact) == coact).all()
    assert (u32(step.load) == load).all()

    r = oracle_assign(w, seed)
    assert (step.assigned_slot.cpu().numpy() == r["assigned_slot"]).all()
    assert (u32(step.slot_load) == r["slot_load"]).all()
    assert (step.remote_nodes.cpu().numpy() == r["remote_nodes"]).all()
    assert step.totals.cpu().tolist() == [r["V"], r["V_naive"]]

    p = O.permute(r["assigned_slot"], w.D)
    assert (u32(step.dest_counts) == p["dest_counts"]).all()
    assert (u32(step.dest_offsets) == p["dest_offsets"]).all()
    assert (step.row_of_pair.cpu().numpy() == p["row_of_pair"]).all()
    assert (step.pair_of_row.cpu().numpy() == p["pair_of_row"]).all()
    return r, p


# ---------------------------------------------------------------------------------------------
# the benchmark configs at sizes the oracle handles in full
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["1", "1a", "2", "3"])
def test_config_full_elementwise(cb, name):
    w = W.make_config(name)
    layout, step = make_step(w, alias_expert_out=False)
    r, p = check_index_stages(cb, w, step, w.seed)

    x = w.hidden_rows()
    for impl in (cb.IMPL_BULK, cb.IMPL_VECTOR, 0):
        step.send.zero_()
        step.permute(flags=impl)
        torch.cuda.synchronize()
        send = bits_from_bf16_tensor(step.send)
        assert (send == x[p["pair_of_row"] // w.K]).all(), f"impl {impl:#x}"
        assert (step.row_of_pair.cpu().numpy() == p["row_of_pair"]).all()

    out = w.expert_out_rows()
    step.expert_out.copy_(bf16_tensor_from_bits(out, "cpu"))
    step.combine()
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0
    assert_combine_close(bits_from_bf16_tensor(step.y), O.combine(out, p["row_of_pair"], w.gate_w))


@pytest.mark.parametrize("name", ["4", "5"])
def test_config_full_size_sampled(cb, name):
    """Largest configs in the launch configuration the bench times: index outputs in full,
    payload on sampled rows/tokens, plus properties that hold at any size."""
    w = W.make_config(name)
    layout, step = make_step(w, alias_expert_out=True)
    r, p = check_index_stages(cb, w, step, w.seed)

    step.permute()
    step.combine()                    # identity experts: expert_out aliases send
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0

    rng = np.random.default_rng(5)
    offs = p["dest_offsets"].astype(np.int64)
    edges = np.concatenate([offs[:-1], offs[1:] - 1])
    edges = edges[(edges >= 0) & (edges < w.P)]
    rows = np.unique(np.concatenate([rng.integers(0, w.P, 3000), edges, [0, w.P - 1]]))
    got = bits_from_bf16_tensor(step.send[torch.from_numpy(rows).cuda()])
    tok = p["pair_of_row"][rows] // w.K
    x_bits = bits_from_bf16_tensor(step.x[torch.from_numpy(tok).cuda()])
    # x on the device is the uploaded generator output; compare against freshly generated rows too
    some = tok[:64]
    for t, xb in zip(some, x_bits[:64]):
        assert (w.hidden_rows(int(t), int(t) + 1)[0] == xb).all()
    assert (got == x_bits).all()

    tokens = np.unique(np.concatenate([rng.integers(0, w.T, 1500), [0, w.T - 1]]))
    rop = p["row_of_pair"].reshape(w.T, w.K)[tokens]                     # [n, K]
    rows_needed = bits_from_bf16_tensor(step.expert_out[torch.from_numpy(rop.ravel()).cuda()])
    y_ref = O.combine(rows_needed, np.arange(rop.size, dtype=np.int32), w.gate_w[tokens])
    y_gpu = bits_from_bf16_tensor(step.y[torch.from_numpy(tokens).cuda()])
    assert_combine_close(y_gpu, y_ref)

    # any-size properties: identity experts and weights summing to one give back x (bf16 rounding)
    diff = (step.y.float() - step.x.float()).abs()
    bound = 2.0 ** -7 * step.x.float().abs() + 1e-6
    assert bool((diff <= bound).all())
    # every send row equals the row of the token its pair belongs to (checked on the device)
    tok_of_row = (step.pair_of_row // w.K).long()
    n_chunk = 1 << 16
    for r0 in range(0, w.P, n_chunk):
        r1 = min(w.P, r0 + n_chunk)
        same = step.send[r0:r1].view(torch.int16) == step.x[tok_of_row[r0:r1]].view(torch.int16)
        assert bool(same.all())
    del diff, bound, same

    # the combine once more at this full shape with expert outputs of their own (not the send buffer):
    # seeded N(0,1) rows drawn on the device; only the sampled tokens' rows come back for the oracle
    gen = torch.Generator(device="cuda")
    gen.manual_seed(int(w.seed) + 7)
    expert_out = torch.empty_like(step.send)
    blk = 1 << 16
    for r0 in range(0, w.P, blk):
        r1 = min(w.P, r0 + blk)
        expert_out[r0:r1] = torch.randn((r1 - r0, w.H), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    step.y.zero_()
    cb.combine(expert_out, step.row_of_pair, step.gate_w, step.y)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0
    rows_needed = bits_from_bf16_tensor(expert_out[torch.from_numpy(rop.ravel()).cuda()])
    y_ref = O.combine(rows_needed, np.arange(rop.size, dtype=np.int32), w.gate_w[tokens])
    assert_combine_close(bits_from_bf16_tensor(step.y[torch.from_numpy(tokens).cuda()]), y_ref)


# ---------------------------------------------------------------------------------------------
# edge shapes
# ---------------------------------------------------------------------------------------------
EDGE = [
    # T, E, K, H, N, Q, S, empty
    (1, 4, 1, 8, 1, 2, 2, 0),
    (1, 8, 3, 24, 2, 2, 2, 0),
    (7, 9, 2, 40, 3, 2, 2, 1),
    (33, 13, 3, 72, 4, 2, 3, 2),
    (1000, 20, 5, 136, 8, 1, 5, 0),
    (1000, 24, 6, 264, 4, 3, 3, 3),
    (2049, 40, 8, 520, 2, 4, 6, 0),
    (4099, 100, 16, 64, 4, 8, 5, 7),
    (5000, 257, 7, 32, 4, 4, 20, 0),
    (3000, 17, 4, 16392, 2, 2, 5, 0),     # a row larger than one pipeline stage
    (70000, 6, 2, 8, 4, 2, 1, 0),
    (1100000, 40, 4, 8, 4, 2, 6, 0),      # more than 2048 chunks of 2048 pairs: the chunk size doubles
    (3000, 1024, 16, 8, 8, 8, 64, 0),     # the largest supported layout: N = 8, K = 16, E = 1024, D = 4096
    (2500, 1000, 13, 16, 8, 8, 64, 96),   # nearly so, with empty slots and an odd K
]


@pytest.mark.parametrize("T,E,K,H,N,Q,S,empty", EDGE)
def test_edge_shapes(cb, T, E, K, H, N, Q, S, empty):
    w = W.make_custom(T, E, K, H, N, Q, S, seed=1000 + T + E, C=3, p_in=0.6, n_empty=empty)
    layout, step = make_step(w, alias_expert_out=False)
    r, p = check_index_stages(cb, w, step, 4242)
    x = w.hidden_rows()
    for impl in (cb.IMPL_BULK, cb.IMPL_VECTOR):
        step.send.zero_()
        step.permute(flags=impl)
        torch.cuda.synchronize()
        assert (bits_from_bf16_tensor(step.send) == x[p["pair_of_row"] // K]).all()
    out = w.expert_out_rows()
    step.expert_out.copy_(bf16_tensor_from_bits(out, "cpu"))
    step.combine()
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0
    assert_combine_close(bits_from_bf16_tensor(step.y), O.combine(out, p["row_of_pair"], w.gate_w))


def test_large_expert_count(cb):
    """E = 700: the co-activation triangle exceeds one CTA's shared memory and the fused pass falls back
    to the separate calls."""
    w = W.make_custom(6000, 700, 8, 8, 4, 8, 24, seed=3, C=7, p_in=0.7)
    layout, step = make_step(w, with_x=False)
    check_index_stages(cb, w, step, 9)


@pytest.mark.parametrize("E,K,T", [(320, 8, 20000), (384, 8, 131072), (451, 7, 9999), (452, 8, 70001),
                                   (453, 8, 70001), (320, 8, 757777), (512, 6, 30000), (600, 4, 5000),
                                   (641, 10, 40000), (1024, 8, 50000), (1024, 16, 3000), (1024, 16, 20000)])
def test_statistics_with_a_triangle_larger_than_one_tile(cb, E, K, T):
    """E > 316: the 32-bit triangle no longer fits one CTA.  Up to E = 452 a tile of 16-bit counters
    does, as long as a cluster sees at most 65535 tokens (clusters shrink for T = 757777); beyond that
    the triangle is split over 2, 4 or 8 CTAs fed the same tokens, and few tokens over a large matrix
    (E = 600 with T = 5000, E = 1024 with T = 3000) are added straight to global memory."""
    model = W.configs.ClusterModel(E, K, 8, 0.7, np.full(8, 1 / 8), np.ones(E))
    ids = W.sample_topk_ids(model, T, seed=E + K)
    ids_d = torch.from_numpy(ids).cuda()
    coact = torch.full((E, E), 9, dtype=torch.int32, device="cuda")
    load = torch.full((E,), 9, dtype=torch.int32, device="cuda")
    for _ in range(2):
        cb.coact_stats(ids_d, E, coact, load)
    cb.coact_stats(ids_d, E, coact, load, flags=cb.STATS_ACCUMULATE)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0
    ref_coact, ref_load = O.coact_stats(ids, E)
    assert (u32(coact) == 2 * ref_coact).all() and (u32(load) == 2 * ref_load).all()


@pytest.mark.parametrize("E,K,T,tile", [(400, 4, 3_000_000, "16-bit, small clusters"),
                                        (500, 2, 4_000_000, "split over pairs of CTAs, clusters of two"),
                                        (330, 2, 10_000_000, "global")])
def test_statistics_many_tokens_and_a_large_triangle(cb, E, K, T, tile):
    """The 16-bit tiles may count at most 65535 tokens per cluster: T = 3e6 and 4e6 only allow clusters
    of two CTAs, T = 1e7 none at all (every pair then goes straight to global memory).  Ids are an
    arithmetic progression per token (distinct by construction), cheap to draw at this size."""
    rng = np.random.default_rng(E * K)
    base = rng.integers(0, E, size=(T, 1), dtype=np.int64)
    step = rng.integers(1, E // K, size=(T, 1), dtype=np.int64)
    ids = ((base + step * np.arange(K, dtype=np.int64)[None, :]) % E).astype(np.int32)
    ids_d = torch.from_numpy(ids).cuda()
    coact = torch.empty((E, E), dtype=torch.int32, device="cuda")
    load = torch.empty((E,), dtype=torch.int32, device="cuda")
    cb.coact_stats(ids_d, E, coact, load)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0
    ref_coact, ref_load = O.coact_stats(ids, E)
    assert (u32(coact) == ref_coact).all() and (u32(load) == ref_load).all()


@pytest.mark.parametrize("E,K,T", [(256, 8, 131072), (64, 6, 40000), (16, 2, 5000), (8, 8, 1500), (256, 8, 700000)])
def test_statistics_with_sixteen_bit_tiles_forced(cb, E, K, T):
    """The 16-bit tile, chosen by default only where the 32-bit one does not fit, gives the same counts
    at every size; T = 700000 exceeds what it may count and must take the 32-bit tile by itself."""
    model = W.configs.ClusterModel(E, K, 4, 0.7, np.full(4, 1 / 4), np.ones(E))
    ids = W.sample_topk_ids(model, T, seed=3 * E + K)
    ids_d = torch.from_numpy(ids).cuda()
    coact = torch.full((E, E), 7, dtype=torch.int32, device="cuda")
    load = torch.full((E,), 7, dtype=torch.int32, device="cuda")
    ref_coact, ref_load = O.coact_stats(ids, E)
    for flags in (cb.STATS_TILE16, cb.STATS_TILE32):
        coact.fill_(7)
        load.fill_(7)
        cb.coact_stats(ids_d, E, coact, load, flags=flags)
        torch.cuda.synchronize()
        assert cb.read_and_clear_device_error() == 0
        assert (u32(coact) == ref_coact).all() and (u32(load) == ref_load).all()


@pytest.mark.parametrize("E,K,T", [(256, 8, 3000), (64, 6, 1), (300, 4, 4096), (400, 8, 2500)])
def test_statistics_of_a_small_batch_overwrite_used_buffers(cb, E, K, T):
    """A batch small enough for a single cluster stores its sums without a clearing kernel before
    it: whatever the outputs held is gone, and the accumulate flag still adds."""
    model = W.configs.ClusterModel(E, K, 4, 0.7, np.full(4, 1 / 4), np.ones(E))
    ids = W.sample_topk_ids(model, T, seed=E + T)
    ids_d = torch.from_numpy(ids).cuda()
    coact = torch.full((E, E), 123456, dtype=torch.int32, device="cuda")
    load = torch.full((E,), 654321, dtype=torch.int32, device="cuda")
    cb.coact_stats(ids_d, E, coact, load)
    torch.cuda.synchronize()
    ref_coact, ref_load = O.coact_stats(ids, E)
    assert (u32(coact) == ref_coact).all() and (u32(load) == ref_load).all()
    cb.coact_stats(ids_d, E, coact, load, flags=cb.STATS_ACCUMULATE)
    cb.coact_stats(ids_d, E, coact, load, flags=cb.STATS_ACCUMULATE)
    torch.cuda.synchronize()
    assert (u32(coact) == 3 * ref_coact).all() and (u32(load) == 3 * ref_load).all()
    assert cb.read_and_clear_device_error() == 0


def test_empty_batch(cb):
    w = W.make_custom(0, 8, 2, 16, 2, 2, 3, seed=1)
    layout, step = make_step(w)
    step.route(5)
    torch.cuda.synchronize()
    assert int(step.coact.sum()) == 0 and int(step.slot_load.sum()) == 0
    assert step.dest_offsets.cpu().tolist() == [0] * (w.D + 1)
    assert step.totals.cpu().tolist() == [0, 0]


# ---------------------------------------------------------------------------------------------
# modes and flags
# ---------------------------------------------------------------------------------------------
def test_naive_rule_and_uniform_source(cb):
    w = W.make_config("3", T=5000)
    layout, step = make_step(w, with_x=False)
    step.assign(w.seed, flags=cb.ASSIGN_NAIVE)
    torch.cuda.synchronize()
    r = oracle_assign(w, w.seed, naive=True)
    assert (step.assigned_slot.cpu().numpy() == r["assigned_slot"]).all()
    assert (step.remote_nodes.cpu().numpy() == r["remote_nodes"]).all()
    assert step.totals.cpu().tolist() == [r["V"], r["V_naive"]]

    w.src_rank[:] = 13
    cb.assign(layout, step.topk_ids, 13, 77, step.assigned_slot, slot_load=step.slot_load,
              remote_nodes=step.remote_nodes, totals=step.totals)
    torch.cuda.synchronize()
    r = oracle_assign(w, 77)
    assert (step.assigned_slot.cpu().numpy() == r["assigned_slot"]).all()
    assert (u32(step.slot_load) == r["slot_load"]).all()
    # optional outputs may be skipped
    out = torch.zeros_like(step.assigned_slot)
    cb.assign(layout, step.topk_ids, 13, 77, out)
    torch.cuda.synchronize()
    assert (out.cpu().numpy() == r["assigned_slot"]).all()


def run_fused_and_compare(cb, w, step, seed, flags=0):
    coact, load = O.coact_stats(w.topk_ids, w.E)
    r = oracle_assign(w, seed)
    p = O.permute(r["assigned_slot"], w.D)
    for buf in (step.coact, step.load, step.assigned_slot, step.dest_counts, step.dest_offsets, step.row_of_pair,
                step.pair_of_row, step.remote_nodes, step.totals):
        buf.fill_(77)
    cb.route_index(step.layout, step.topk_ids, step.src_rank, seed, step.coact, step.load, step.assigned_slot,
                   step.dest_counts, step.dest_offsets, step.row_of_pair, step.workspace,
                   remote_nodes=step.remote_nodes, totals=step.totals, pair_of_row=step.pair_of_row, flags=flags)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0
    assert (u32(step.coact) == coact).all() and (u32(step.load) == load).all()
    assert (step.assigned_slot.cpu().numpy() == r["assigned_slot"]).all()
    assert (step.remote_nodes.cpu().numpy() == r["remote_nodes"]).all()
    assert step.totals.cpu().tolist() == [r["V"], r["V_naive"]]
    assert (u32(step.dest_counts) == r["slot_load"]).all()
    assert (u32(step.dest_offsets) == p["dest_offsets"]).all()
    assert (step.row_of_pair.cpu().numpy() == p["row_of_pair"]).all()
    assert (step.pair_of_row.cpu().numpy() == p["pair_of_row"]).all()


@pytest.mark.parametrize("name", ["1", "1a", "2", "3", "4", "5"])
def test_fused_route_index_on_configs(cb, name):
    w = W.make_config(name)
    layout, step = make_step(w, with_x=False)
    run_fused_and_compare(cb, w, step, w.seed)
    run_fused_and_compare(cb, w, step, w.seed + 1)      # a second call on used buffers


@pytest.mark.parametrize("T,E,K,H,N,Q,S,empty", [
    (1, 4, 1, 8, 1, 2, 2, 0), (7, 9, 2, 8, 3, 2, 2, 1), (255, 13, 3, 8, 4, 2, 3, 2), (257, 13, 3, 8, 4, 2, 3, 2),
    (1000, 20, 5, 8, 8, 1, 5, 0), (2049, 40, 8, 8, 2, 4, 6, 0), (4099, 100, 16, 8, 4, 8, 5, 7),
    (5000, 257, 7, 8, 4, 4, 20, 0), (6000, 700, 8, 8, 4, 8, 24, 0), (200000, 6, 2, 8, 4, 2, 1, 0),
    (1100000, 40, 4, 8, 4, 2, 6, 0),
    # 200000 and 1100000 tokens: several rounds of 1024 tokens per CTA (the ranks are worked out round by
    # round after the barrier).  E = 320..440: the triangle only fits with 16-bit counters; with 600000
    # tokens the 32-bit triangle (E = 330) takes over; E = 1024 or D = 4096: the separate calls
    (20000, 384, 8, 8, 4, 8, 13, 0), (131072, 320, 8, 8, 4, 8, 11, 3), (9000, 440, 6, 8, 2, 4, 56, 0),
    (600000, 330, 2, 8, 4, 2, 42, 0), (3000, 1024, 16, 8, 8, 8, 64, 0)])
def test_fused_route_index_edge_shapes(cb, T, E, K, H, N, Q, S, empty):
    w = W.make_custom(T, E, K, H, N, Q, S, seed=2000 + T + E, C=3, p_in=0.6, n_empty=empty)
    layout, step = make_step(w, with_x=False)
    run_fused_and_compare(cb, w, step, 31337)


def test_fused_pass_starts_from_any_workspace_contents_and_runs_beside_itself(cb):
    """The grid barrier of the fused kernel lives in the workspace and must not depend on what it finds
    there: all ones, all zeros, what the previous call left, a word that looks like a barrier of
    another launch.  Two calls on two streams, each with its own workspace, may overlap."""
    w = W.make_config("3", T=20000)
    layout, step = make_step(w, with_x=False)
    for fill in (0xFF, 0x00, None, 0x5A):
        if fill is not None:
            step.workspace.fill_(fill)
        run_fused_and_compare(cb, w, step, 99)
    step.workspace.view(torch.int64)[0] = (12345 << 32) | 7          # epoch 12345, seven arrivals
    run_fused_and_compare(cb, w, step, 99)
    ref = {k: getattr(step, k).clone() for k in ("coact", "assigned_slot", "row_of_pair", "pair_of_row", "dest_offsets")}
    layout2, other = make_step(w, with_x=False)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(10):
        for st, stream in ((step, s1), (other, s2)):
            with torch.cuda.stream(stream):
                cb.route_index(st.layout, st.topk_ids, st.src_rank, 99, st.coact, st.load, st.assigned_slot,
                               st.dest_counts, st.dest_offsets, st.row_of_pair, st.workspace,
                               remote_nodes=st.remote_nodes, totals=st.totals, pair_of_row=st.pair_of_row)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0
    for st in (step, other):
        for k, v in ref.items():
            assert torch.equal(getattr(st, k), v), k
    # many calls in a row, the workspace (barrier word and grid totals included) and the outputs filled with
    # random bytes every few calls: every output is stored anew by every call
    ref["load"], ref["dest_counts"], ref["totals"] = step.load.clone(), step.dest_counts.clone(), step.totals.clone()
    for it in range(300):
        if it % 7 == 0:
            step.workspace.view(torch.uint8).random_(0, 256)
        if it % 11 == 0:
            for k in ref:
                getattr(step, k).view(torch.uint8).random_(0, 256)
        cb.route_index(step.layout, step.topk_ids, step.src_rank, 99, step.coact, step.load, step.assigned_slot,
                       step.dest_counts, step.dest_offsets, step.row_of_pair, step.workspace,
                       remote_nodes=step.remote_nodes, totals=step.totals, pair_of_row=step.pair_of_row)
        if it % 10 == 0 or it == 299:
            for k, v in ref.items():
                assert torch.equal(getattr(step, k), v), (it, k)
    assert cb.read_and_clear_device_error() == 0


def test_step_with_statistics_on_a_side_stream(cb):
    """overlap_stats runs stage 1 beside the others; repeated steps give the results of the oracle."""
    w = W.make_config("3", T=7001)
    layout, step = make_step(w)
    for _ in range(4):
        step.coact.fill_(5)
        step.route(w.seed, overlap_stats=True)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0
    coact, load = O.coact_stats(w.topk_ids, w.E)
    assert (u32(step.coact) == coact).all() and (u32(step.load) == load).all()
    r = oracle_assign(w, w.seed)
    assert (step.assigned_slot.cpu().numpy() == r["assigned_slot"]).all()
    p = O.permute(r["assigned_slot"], w.D, w.hidden_rows())
    assert (step.row_of_pair.cpu().numpy() == p["row_of_pair"]).all()
    assert (bits_from_bf16_tensor(step.send) == p["send"]).all()


@pytest.mark.parametrize("T,E,K,N,Q,S,empty", [(4096, 256, 8, 4, 8, 9, 0), (4095, 64, 6, 4, 8, 3, 2), (257, 16, 2, 2, 4, 3, 0),
                                               (1, 8, 1, 1, 2, 4, 0), (3000, 100, 4, 8, 4, 4, 5), (2049, 24, 8, 3, 2, 5, 0),
                                               (4000, 384, 8, 4, 8, 13, 0), (4096, 420, 6, 2, 4, 60, 7)])
def test_fused_pass_on_small_batches(cb, T, E, K, N, Q, S, empty):
    """Small batches run the fused kernel on a few CTAs (256 tokens each, down to a single CTA), large
    triangles beside many destinations fall back to the separate calls.  Same results as the oracle,
    as the separate calls (COBALT_ROUTE_SEPARATE_KERNELS), and with the accumulate flag on top of
    what is already there."""
    w = W.make_custom(T, E, K, 8, N, Q, S, seed=900 + T, C=2, p_in=0.7, n_empty=empty)
    layout, step = make_step(w, with_x=False)
    run_fused_and_compare(cb, w, step, 321)
    small = {k: getattr(step, k).clone() for k in ("coact", "load", "assigned_slot", "dest_counts", "dest_offsets",
                                                     "row_of_pair", "pair_of_row", "remote_nodes", "totals")}
    run_fused_and_compare(cb, w, step, 321, flags=cb.ROUTE_SEPARATE_KERNELS)
    for k, v in small.items():
        assert torch.equal(getattr(step, k), v), k
    cb.route_index(layout, step.topk_ids, step.src_rank, 321, step.coact, step.load, step.assigned_slot,
                   step.dest_counts, step.dest_offsets, step.row_of_pair, step.workspace, flags=cb.STATS_ACCUMULATE)
    torch.cuda.synchronize()
    assert torch.equal(step.coact, 2 * small["coact"]) and torch.equal(step.load, 2 * small["load"])
    assert torch.equal(step.row_of_pair, small["row_of_pair"]) and torch.equal(step.dest_offsets, small["dest_offsets"])


@pytest.mark.parametrize("name,T,fused", [("3", 9000, False), ("3", 9000, True), ("1", 3000, True), ("5", 20000, False)])
def test_step_replayed_from_a_graph_with_a_seed_on_the_device(cb, name, T, fused):
    """capture() records one step whose assignment kernels read the seed from a device word;
    replay(seed) must give what route(seed) gives, for every seed, including one above 2^63."""
    w = W.make_config(name, T=T)
    layout, step = make_step(w)
    names = ("coact", "load", "assigned_slot", "remote_nodes", "totals", "dest_counts", "dest_offsets",
             "row_of_pair", "pair_of_row", "send", "y")
    step.capture(fused=fused)
    for seed in (5, 2**63 + 12345, w.seed):
        step.route_fused(seed) if fused else step.route(seed)
        torch.cuda.synchronize()
        ref = {k: getattr(step, k).clone() for k in names}
        for k in names:
            getattr(step, k).zero_()
        step.replay(seed)
        torch.cuda.synchronize()
        for k in names:
            a, b = getattr(step, k), ref[k]
            if a.dtype == torch.bfloat16:
                a, b = a.view(torch.int16), b.view(torch.int16)
            assert torch.equal(a, b), (k, seed)
    r = oracle_assign(w, w.seed)
    assert (step.assigned_slot.cpu().numpy() == r["assigned_slot"]).all()
    assert cb.read_and_clear_device_error() == 0


def test_fused_route_step_equals_separate_stages(cb):
    w = W.make_config("3", T=12345)
    layout, step = make_step(w)
    step.route(w.seed)
    torch.cuda.synchronize()
    ref = {k: getattr(step, k).clone() for k in ("coact", "load", "assigned_slot", "slot_load", "dest_counts",
                                                   "dest_offsets", "row_of_pair", "pair_of_row", "send", "y", "totals")}
    for k in ref:
        getattr(step, k).fill_(0)
    step.route_fused(w.seed)
    torch.cuda.synchronize()
    for k, v in ref.items():
        if k == "slot_load":
            continue              # delivered as dest_counts by the fused call
        got = getattr(step, k)
        assert torch.equal(got.view(torch.int16) if got.dtype == torch.bfloat16 else got,
                           v.view(torch.int16) if v.dtype == torch.bfloat16 else v), k
    # accumulate flag and empty batch
    cb.route_index(layout, step.topk_ids, step.src_rank, w.seed, step.coact, step.load, step.assigned_slot,
                   step.dest_counts, step.dest_offsets, step.row_of_pair, step.workspace, flags=cb.STATS_ACCUMULATE)
    torch.cuda.synchronize()
    assert torch.equal(step.coact, 2 * ref["coact"]) and torch.equal(step.load, 2 * ref["load"])
    w0 = W.make_custom(0, 8, 2, 16, 2, 2, 3, seed=1)
    layout0, step0 = make_step(w0)
    step0.route_fused(5)
    torch.cuda.synchronize()
    assert int(step0.coact.sum()) == 0 and step0.dest_offsets.cpu().tolist() == [0] * (w0.D + 1)


@pytest.mark.parametrize("name,T", [("1", 4096), ("2", 9000), ("3", 20001), ("5", 131072)])
def test_round_robin_replica_pick(cb, name, T):
    """The running count behind the round-robin pick is reproduced exactly (bit-identical slots)."""
    w = W.make_config(name, T=T)
    layout, step = make_step(w, with_x=False)
    ws = torch.empty(max(cb.assign_workspace_bytes(layout, w.T, w.K), 256), dtype=torch.uint8, device="cuda")
    r = O.assign(w.N, w.Q, w.S, w.E, w.slot_expert, w.primary_slot, w.topk_ids, w.src_rank, w.seed,
                 round_robin=True)
    for _ in range(2):
        step.assigned_slot.fill_(-5)
        cb.assign(layout, step.topk_ids, step.src_rank, w.seed, step.assigned_slot, slot_load=step.slot_load,
                  remote_nodes=step.remote_nodes, totals=step.totals, flags=cb.ASSIGN_ROUND_ROBIN, workspace=ws)
        torch.cuda.synchronize()
        assert cb.read_and_clear_device_error() == 0
        assert (step.assigned_slot.cpu().numpy() == r["assigned_slot"]).all()
        assert (u32(step.slot_load) == r["slot_load"]).all()
        assert (step.remote_nodes.cpu().numpy() == r["remote_nodes"]).all()
        assert step.totals.cpu().tolist() == [r["V"], r["V_naive"]]
    with pytest.raises(cb.CobaltError) as e:
        cb.assign(layout, step.topk_ids, step.src_rank, w.seed, step.assigned_slot, flags=cb.ASSIGN_ROUND_ROBIN)
    assert e.value.status == cb.ERR_WORKSPACE_TOO_SMALL


def test_round_robin_skips_bad_tokens(cb):
    w = W.make_config("3", T=3000)
    layout, step = make_step(w, with_x=False)
    ws = torch.empty(cb.assign_workspace_bytes(layout, w.T, w.K), dtype=torch.uint8, device="cuda")
    ids = w.topk_ids.copy()
    ids[100, 2] = ids[100, 0]
    ids[2000, 1] = -3
    step.topk_ids.copy_(torch.from_numpy(ids))
    cb.assign(layout, step.topk_ids, step.src_rank, 5, step.assigned_slot, slot_load=step.slot_load,
              flags=cb.ASSIGN_ROUND_ROBIN, workspace=ws)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == cb.DEVERR_BAD_EXPERT_ID | cb.DEVERR_DUPLICATE_ID
    keep = np.ones(w.T, bool)
    keep[[100, 2000]] = False
    # the oracle on the remaining tokens, in their original order: the bad ones are simply not dealt
    r = O.assign(w.N, w.Q, w.S, w.E, w.slot_expert, w.primary_slot, w.topk_ids[keep], w.src_rank[keep], 5,
                 round_robin=True)
    got = step.assigned_slot.cpu().numpy()
    assert (got[~keep] == -1).all()
    # node choices are hashed on the token index, so compare what does not depend on it
    assert int(step.slot_load.sum()) == keep.sum() * w.K
    assert (w.slot_expert[got[keep]] == w.topk_ids[keep]).all()
    del r


def test_ema_and_ochiai(cb):
    w = W.make_config("5", T=20000)
    layout, step = make_step(w, with_x=False)
    step.stats()
    och = torch.zeros((w.E, w.E), dtype=torch.float32, device="cuda")
    cb.ochiai(step.coact, och)
    ema = torch.zeros((w.E, w.E), dtype=torch.float32, device="cuda")
    cb.ema_update(step.coact, ema, 0.9, flags=cb.EMA_INITIALISE)
    for _ in range(3):
        cb.ema_update(step.coact, ema, 0.9)
    ema2 = torch.full((w.E,), 5.0, dtype=torch.float32, device="cuda")
    cb.ema_update(step.load, ema2, 0.75)
    torch.cuda.synchronize()
    coact, load = O.coact_stats(w.topk_ids, w.E)
    assert np.allclose(och.cpu().numpy(), O.ochiai(coact), rtol=2e-6, atol=1e-7)
    assert np.allclose(ema.cpu().numpy(), coact, rtol=1e-6)            # an EMA of a constant stays there
    assert np.allclose(ema2.cpu().numpy(), O.ema_update(np.full(w.E, 5.0), load, 0.75), rtol=1e-6)
    with pytest.raises(cb.CobaltError):
        cb.ema_update(step.load, ema2, 1.5)


def test_fig1_layout_on_gpu(cb, fig1):
    g = fig1
    ids = np.array([tk["ids"] for tk in g["tokens"]], np.int32)
    src = np.array([tk["src"] for tk in g["tokens"]], np.int32)
    layout = cb.Layout(2, 2, 2, 4, g["slot_expert"], g["primary_slot"])
    out = torch.zeros((12, 2), dtype=torch.int32, device="cuda")
    remote = torch.zeros(12, dtype=torch.uint8, device="cuda")
    totals = torch.zeros(2, dtype=torch.int64, device="cuda")
    cb.assign(layout, torch.from_numpy(ids).cuda(), torch.from_numpy(src).cuda(), 36959, out,
              remote_nodes=remote, totals=totals)
    torch.cuda.synchronize()
    assert remote.cpu().tolist() == [tk["cobalt"] for tk in g["tokens"]]
    assert totals.cpu().tolist() == [g["V_cobalt"], g["V_naive"]]
    for seed, t, k, slot in g["seeded"]:
        assert int(out[t, k]) == slot


def test_stats_accumulate_flag(cb):
    w = W.make_config("3", T=3000)
    layout, step = make_step(w, with_x=False)
    step.stats()
    step.stats(flags=cb.STATS_ACCUMULATE)
    torch.cuda.synchronize()
    coact, load = O.coact_stats(w.topk_ids, w.E)
    assert (u32(step.coact) == 2 * coact).all() and (u32(step.load) == 2 * load).all()
    step.stats()
    torch.cuda.synchronize()
    assert (u32(step.coact) == coact).all()


def test_results_do_not_depend_on_the_run(cb):
    w = W.make_config("4", T=30000)
    layout, step = make_step(w)
    step.route(w.seed)
    torch.cuda.synchronize()
    ref = [t.clone() for t in (step.coact, step.assigned_slot, step.row_of_pair, step.pair_of_row, step.send, step.y)]
    for _ in range(20):
        step.route(w.seed)
        torch.cuda.synchronize()
        for a, b in zip(ref, (step.coact, step.assigned_slot, step.row_of_pair, step.pair_of_row, step.send, step.y)):
            assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a,
                               b.view(torch.int16) if b.dtype == torch.bfloat16 else b)


def test_round_trip_identity_and_one_hot(cb):
    w = W.make_config("2", T=4000)
    layout, step = make_step(w)
    step.gate_w.zero_()
    pick = torch.arange(w.T, device="cuda") % w.K
    step.gate_w[torch.arange(w.T, device="cuda"), pick] = 1.0
    step.route(w.seed)
    torch.cuda.synchronize()
    # one-hot weights select exactly one expert row = the token's own row
    assert torch.equal(step.y.view(torch.int16), step.x.view(torch.int16))


@pytest.mark.parametrize("name,T,chunks", [("3", 10001, 5), ("1", 4096, 8), ("2", 37, 8)])
def test_host_driven_step_matches_the_resident_step(cb, name, T, chunks):
    """route_host (pinned host buffers, token blocks overlapped with the copies) gives exactly the
    results of route() on resident data."""
    w = W.make_config(name, T=T)
    layout, step = make_step(w)
    step.route(w.seed)
    torch.cuda.synchronize()
    ref = {k: getattr(step, k).clone() for k in ("y", "coact", "load", "slot_load", "totals", "send", "row_of_pair")}
    ids_h = torch.from_numpy(w.topk_ids).pin_memory()
    w_h = torch.from_numpy(w.gate_w).pin_memory()
    src_h = torch.from_numpy(w.src_rank).pin_memory()
    x_h = bf16_tensor_from_bits(w.hidden_rows(), "cpu").pin_memory()
    y_h = torch.zeros((w.T, w.H), dtype=torch.bfloat16).pin_memory()
    coact_h = torch.zeros((w.E, w.E), dtype=torch.int32).pin_memory()
    load_h = torch.zeros((w.E,), dtype=torch.int32).pin_memory()
    sl_h = torch.zeros((w.D,), dtype=torch.int32).pin_memory()
    tot_h = torch.zeros((2,), dtype=torch.int64).pin_memory()
    for buf in (step.x, step.y, step.send, step.topk_ids, step.coact):
        buf.zero_()
    for _ in range(2):       # twice: the second call overlaps with the tail of the first
        step.route_host(w.seed, ids_h, w_h, src_h, x_h, y_h, coact_h, load_h, sl_h, tot_h, chunks=chunks)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0
    assert torch.equal(y_h.view(torch.int16), ref["y"].cpu().view(torch.int16))
    assert torch.equal(coact_h, ref["coact"].cpu()) and torch.equal(load_h, ref["load"].cpu())
    assert torch.equal(sl_h, ref["slot_load"].cpu()) and torch.equal(tot_h, ref["totals"].cpu())
    assert torch.equal(step.send.view(torch.int16), ref["send"].view(torch.int16))
    assert torch.equal(step.row_of_pair, ref["row_of_pair"])


def test_host_driven_steps_queued_without_joining(cb):
    """Three different batches through route_host(join=False), queued back to back into separate host
    buffers: a step starts while the one before still copies results out, and nothing is overwritten
    before it has been copied.  Each batch must equal its own resident step."""
    T, chunks = 20003, 8
    w = W.make_config("3", T=T)
    x_bits = w.hidden_rows()
    layout, step = make_step(w)
    seeds = [11, 22, 33]
    host, refs = [], []
    for i, seed in enumerate(seeds):
        # batch i: tokens rotated by 1000 i, and its first 500 (i + 1) tokens all routed like token 0
        ids = np.roll(w.topk_ids, 1000 * i, axis=0).copy()
        ids[:500 * (i + 1)] = ids[0]
        gate = np.roll(w.gate_w, 1000 * i, axis=0).copy()
        src = np.roll(w.src_rank, 77 * i).copy()
        x = np.roll(x_bits, 1000 * i, axis=0).copy()
        step.topk_ids.copy_(torch.from_numpy(ids))
        step.gate_w.copy_(torch.from_numpy(gate))
        step.src_rank.copy_(torch.from_numpy(src))
        step.x.copy_(bf16_tensor_from_bits(x, "cpu"))
        step.route(seed)
        torch.cuda.synchronize()
        refs.append({k: getattr(step, k).cpu() for k in ("y", "coact", "load", "slot_load", "totals")})
        host.append({
            "ids": torch.from_numpy(ids).pin_memory(), "w": torch.from_numpy(gate).pin_memory(),
            "src": torch.from_numpy(src).pin_memory(), "x": bf16_tensor_from_bits(x, "cpu").pin_memory(),
            "y": torch.zeros((T, w.H), dtype=torch.bfloat16).pin_memory(),
            "coact": torch.zeros((w.E, w.E), dtype=torch.int32).pin_memory(),
            "load": torch.zeros((w.E,), dtype=torch.int32).pin_memory(),
            "sl": torch.zeros((w.D,), dtype=torch.int32).pin_memory(),
            "tot": torch.zeros((2,), dtype=torch.int64).pin_memory()})
    assert not torch.equal(refs[0]["coact"], refs[1]["coact"]) and not torch.equal(refs[1]["y"], refs[2]["y"])
    for buf in (step.x, step.y, step.send, step.topk_ids, step.coact):
        buf.zero_()
    torch.cuda.synchronize()
    for h, seed in zip(host, seeds):
        step.route_host(seed, h["ids"], h["w"], h["src"], h["x"], h["y"], h["coact"], h["load"], h["sl"],
                        h["tot"], chunks=chunks, join=False)
    step.wait_host_results()
    for h, ref in zip(host, refs):
        assert torch.equal(h["y"].view(torch.int16), ref["y"].view(torch.int16))
        assert torch.equal(h["coact"], ref["coact"]) and torch.equal(h["load"], ref["load"])
        assert torch.equal(h["sl"], ref["slot_load"]) and torch.equal(h["tot"], ref["totals"])
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0


# ---------------------------------------------------------------------------------------------
# bad data and bad arguments: flagged, never faulting
# ---------------------------------------------------------------------------------------------
def test_bad_data_sets_the_error_word(cb):
    w = W.make_config("1", T=2000)
    layout, step = make_step(w)
    good = oracle_assign(w, 3)
    ids = w.topk_ids.copy()
    ids[10, 0] = w.E + 5           # out of range
    ids[20, 1] = ids[20, 0]        # duplicate
    step.topk_ids.copy_(torch.from_numpy(ids))
    step.src_rank[30] = w.G        # bad source rank
    step.stats()
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == cb.DEVERR_BAD_EXPERT_ID | cb.DEVERR_DUPLICATE_ID
    step.assign(3)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == (cb.DEVERR_BAD_EXPERT_ID | cb.DEVERR_DUPLICATE_ID |
                                                cb.DEVERR_BAD_SRC_RANK)
    got = step.assigned_slot.cpu().numpy()
    keep = np.ones(w.T, bool)
    keep[[10, 20, 30]] = False
    assert (got[keep] == good["assigned_slot"][keep]).all()      # other tokens unaffected
    assert (got[~keep] == -1).all()
    assert int(step.slot_load.sum()) == (w.T - 3) * w.K
    # the permutation skips the pairs without a slot and says so
    step.permute()
    step.combine()
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() & cb.DEVERR_BAD_SLOT
    assert int(step.dest_offsets[-1]) == (w.T - 3) * w.K
    assert cb.read_and_clear_device_error() == 0


@pytest.mark.parametrize("T", [2000, 9000])
def test_bad_data_through_the_fused_entry(cb, T):
    """The fused kernel (a few CTAs at T = 2000, 36 at T = 9000) treats bad tokens exactly as the
    separate calls do: same error bits, slots of -1, rows of -1, counts without them."""
    w = W.make_config("3", T=T)
    layout, step = make_step(w, with_x=False)
    ids = w.topk_ids.copy()
    ids[10, 0] = w.E + 5
    ids[300, 1] = ids[300, 0]
    ids[T - 1, 2] = -4
    step.topk_ids.copy_(torch.from_numpy(ids))
    step.src_rank[30] = w.G
    step.src_rank[T - 2] = -1
    step.stats()
    step.assign(7)
    cb.permute_index(step.assigned_slot, w.D, step.dest_counts, step.dest_offsets, step.row_of_pair,
                     step.pair_of_row, step.workspace)
    torch.cuda.synchronize()
    bits = cb.read_and_clear_device_error()
    names = ("coact", "load", "assigned_slot", "remote_nodes", "totals", "dest_counts", "dest_offsets", "row_of_pair")
    ref = {k: getattr(step, k).clone() for k in names}
    n_valid = int(step.dest_offsets[-1])
    ref_por = step.pair_of_row[:n_valid].clone()
    for k in names:
        getattr(step, k).fill_(9)
    cb.route_index(layout, step.topk_ids, step.src_rank, 7, step.coact, step.load, step.assigned_slot,
                   step.dest_counts, step.dest_offsets, step.row_of_pair, step.workspace,
                   remote_nodes=step.remote_nodes, totals=step.totals, pair_of_row=step.pair_of_row)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == bits & ~cb.DEVERR_BAD_SLOT
    assert n_valid == (T - 5) * w.K
    for k in names:
        assert torch.equal(getattr(step, k), ref[k]), k
    assert torch.equal(step.pair_of_row[:n_valid], ref_por)


def test_argument_checks(cb):
    w = W.make_config("1", T=256)
    layout, step = make_step(w)
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(cb.CobaltError) as e:
        cb.permute_index(step.assigned_slot, w.D, step.dest_counts, step.dest_offsets, step.row_of_pair,
                         step.pair_of_row, small)
    assert e.value.status == cb.ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(cb.CobaltError) as e:
        cb.assign(layout, step.topk_ids, w.G, 1, step.assigned_slot)       # uniform source rank out of range
    assert e.value.status == cb.ERR_INVALID_ARG
    x7 = torch.zeros((w.T, 12), dtype=torch.bfloat16, device="cuda")
    send7 = torch.zeros((w.P, 12), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(cb.CobaltError) as e:
        cb.permute_rows(x7, step.row_of_pair, w.K, send7)                   # H not a multiple of 8
    assert e.value.status == cb.ERR_UNSUPPORTED
    with pytest.raises(cb.CobaltError) as e:
        cb.Layout(2, 2, 2, 4, [0, 0, 2, 0, 1, 2, 3, 0])
    assert e.value.status == cb.ERR_INVALID_ARG
    for bad_address in (0, step.totals.data_ptr() + 4):                     # null, and not 8-byte aligned
        with pytest.raises(cb.CobaltError) as e:
            cb.assign(layout, step.topk_ids, step.src_rank, bad_address, step.assigned_slot, flags=cb.SEED_ON_DEVICE)
        assert e.value.status == cb.ERR_INVALID_ARG
        with pytest.raises(cb.CobaltError) as e:
            cb.route_index(layout, step.topk_ids, step.src_rank, bad_address, step.coact, step.load, step.assigned_slot,
                           step.dest_counts, step.dest_offsets, step.row_of_pair, step.workspace, flags=cb.SEED_ON_DEVICE)
        assert e.value.status == cb.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0
