"""The allocation-free dispatch-index entry point (director_dispatch_index_static).

Callers that are not allowed to allocate device memory - code living inside an engine that owns the
device heap, loops that must never wait on the allocator, processes with a fixed memory reservation -
cannot create a context, because creating one allocates its workspace.  This entry point keeps its
scratch in a fixed array inside the library instead.  The test calls it through the C ABI twice in a
row, on two different batches, and requires bit-identical results to director_dispatch (the existing,
context-based entry point) and to the CPU oracle's permutation, and that the device's free memory does not change across the calls.

The file name makes pytest collect it after every other test file."""
import numpy as np
import pytest

from oracle import director_oracle as orc
from paper_2607_08782_b200 import synth

pytestmark = pytest.mark.gpu


def _replica_tables(X, C_max):
    """rep_start [E+1], rep_slot [sum of replicas]: slot = rank*C_max + position of the expert among the
    rank's hosted experts (ascending id); an expert's replicas in ascending rank order."""
    E, R = X.shape
    pos = np.cumsum(X, axis=0) - 1                 # position of expert e among the experts of rank j
    rep_start, rep_slot = [0], []
    for e in range(E):
        for j in range(R):
            if X[e, j]:
                rep_slot.append(j * C_max + int(pos[e, j]))
        rep_start.append(len(rep_slot))
    return np.array(rep_start, dtype=np.int32), np.array(rep_slot, dtype=np.int32)


def test_static_entry_point_matches_director_dispatch_on_two_calls_in_a_row():
    import torch
    from paper_2607_08782_b200 import binding
    from paper_2607_08782_b200.layer import MoELayer

    E, K, R, C, H, F = 60, 4, 8, 9, 256, 128
    X = synth.placement_from_ranks(np.arange(E) % R, R)
    X[3, 5] = X[3, 6] = X[17, 0] = X[59, 2] = 1           # a few replicas
    rep_start, rep_slot = _replica_tables(X, C)
    dev = "cuda"
    w = torch.zeros((E, F, H), dtype=torch.bfloat16, device=dev)
    wd = torch.zeros((E, H, F), dtype=torch.bfloat16, device=dev)
    layer = MoELayer(3000, H, F, E, K, 0, R, C, w, w, wd, device=dev)
    layer.set_placement(X)
    d_start = torch.from_numpy(rep_start).to(dev)
    d_slot = torch.from_numpy(rep_slot).to(dev)

    for call, (T, seed) in enumerate([(3000, 71), (1237, 72)]):
        shape = synth.Shape("na", T, H, E, K, F, 0, R, C, 1.3, seed)
        logits = torch.from_numpy(synth.make_logits(shape)).to(dev)
        x = torch.zeros((T, H), dtype=torch.bfloat16, device=dev)
        layer.route(T, logits)
        layer.dispatch(T, x)                                   # existing entry point
        A = T * K
        row_token = torch.full((A,), -7, dtype=torch.int32, device=dev)
        inv_row = torch.full((T, K), -7, dtype=torch.int32, device=dev)
        dest_rank = torch.full((T, K), -7, dtype=torch.int32, device=dev)
        seg_offsets = torch.full((R * C + 1,), -7, dtype=torch.int32, device=dev)
        status = torch.zeros((1,), dtype=torch.int32, device=dev)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        binding.dispatch_index_static(T, K, E, R, C, layer.topk_idx, d_start, d_slot, row_token, inv_row,
                                      dest_rank, seg_offsets, status)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        if call > 0:                                           # the first call may load the module's image
            assert free_after == free_before, "the allocation-free entry point changed the free device memory"
        assert int(status.item()) == 0
        assert torch.equal(seg_offsets, layer.seg_offsets), f"call {call}: seg_offsets"
        assert torch.equal(row_token, layer.row_token[:A]), f"call {call}: row_token"
        assert torch.equal(inv_row, layer.inv_row[:T]), f"call {call}: inv_row"
        assert torch.equal(dest_rank, layer.dest_rank[:T]), f"call {call}: dest_rank"
        assert int(seg_offsets[-1]) == A
        # and directly against the CPU oracle's definition of the permutation
        d_o = orc.dispatch(layer.topk_idx[:T].cpu().numpy(), X, C)
        assert np.array_equal(seg_offsets.cpu().numpy(), d_o["seg_offsets"]), f"call {call}: seg_offsets vs oracle"
        assert np.array_equal(row_token.cpu().numpy(), d_o["row_token"]), f"call {call}: row_token vs oracle"
        assert np.array_equal(inv_row.cpu().numpy(), d_o["inv_row"]), f"call {call}: inv_row vs oracle"
        assert np.array_equal(dest_rank.cpu().numpy(), d_o["dest_rank"]), f"call {call}: dest_rank vs oracle"


def test_static_entry_point_rejects_problems_beyond_its_fixed_scratch():
    import torch
    from paper_2607_08782_b200 import binding
    lib = binding.load_library()
    t = torch.zeros((16,), dtype=torch.int32, device="cuda")
    p = t.data_ptr()
    # ceil(T/256) * E must fit the 1 MiB array: 600000 tokens at E = 128 do not
    rc = lib.director_dispatch_index_static(600000, 2, 128, 16, 9, p, p, p, p, p, p, p, None, None)
    assert rc == 9 and "fixed scratch" in binding.status_string(rc)
    assert lib.director_dispatch_index_static(0, 2, 128, 16, 9, p, p, p, p, p, p, p, None, None) == 1
    assert lib.director_dispatch_index_static(64, 2, 128, 16, 9, None, p, p, p, p, p, p, None, None) == 1


def test_static_entry_point_skips_and_flags_a_routed_expert_without_a_replica():
    """Caller-built tables are not trusted: an expert that tokens are routed to but that has no replica in the
    tables is skipped (row -1), DIRECTOR_ERR_BAD_INDEX is raised in the status word, nothing is written out of bounds
    and every other assignment is placed exactly as the oracle places it on the remaining experts."""
    import torch
    from paper_2607_08782_b200 import binding
    E, K, R, C, T = 6, 2, 3, 2, 500
    dev = "cuda"
    rng = np.random.default_rng(5)
    idx = np.stack([rng.permutation(E)[:K] for _ in range(T)]).astype(np.int32)
    X = synth.placement_from_ranks(np.arange(E) % R, R)
    rep_start, rep_slot = _replica_tables(X, C)
    # drop expert 2's only replica from the tables: rep_start keeps its prefix form, expert 2 gets zero replicas
    lo, hi = int(rep_start[2]), int(rep_start[3])
    bad_slot = np.delete(rep_slot, np.arange(lo, hi))
    bad_start = rep_start.copy()
    bad_start[3:] -= (hi - lo)
    d_idx = torch.from_numpy(idx).to(dev)
    A = T * K
    guard = 64                                               # canaries around every output
    bufs = {n: torch.full((size + 2 * guard,), -7, dtype=torch.int32, device=dev)
            for n, size in (("row_token", A), ("inv_row", A), ("dest_rank", A), ("seg", R * C + 1))}
    view = {n: b[guard:-guard] for n, b in bufs.items()}
    status = torch.zeros((1,), dtype=torch.int32, device=dev)
    binding.dispatch_index_static(T, K, E, R, C, d_idx, torch.from_numpy(bad_start).to(dev),
                                  torch.from_numpy(bad_slot).to(dev), view["row_token"], view["inv_row"].view(T, K),
                                  view["dest_rank"].view(T, K), view["seg"], status)
    torch.cuda.synchronize()
    assert int(status.item()) == 7                           # DIRECTOR_ERR_BAD_INDEX
    for n, b in bufs.items():                                # nothing outside the arrays was touched
        assert bool((b[:guard] == -7).all()) and bool((b[-guard:] == -7).all()), n
    inv = view["inv_row"].view(T, K).cpu().numpy()
    hit = idx == 2
    assert (inv[hit] == -1).all() and (inv[~hit] >= 0).all()
    assert int(view["seg"][-1]) == int((~hit).sum())
    # the remaining assignments: same rows as the oracle gives when expert 2's choices are routed nowhere, i.e. the
    # permutation of the other experts' assignments is unchanged by the hole
    rows = inv[~hit]
    assert len(np.unique(rows)) == len(rows) and rows.max() == len(rows) - 1
    rt = view["row_token"].cpu().numpy()[:len(rows)]
    tok = np.repeat(np.arange(T), K).reshape(T, K)[~hit]
    assert np.array_equal(rt[rows], tok)
