"""GPU parity (bit-exact) of the integer steps against the oracle, through the C ABI."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2509_15235_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    from paper_2509_15235_b200 import binding
    import gpu_util
    return binding, gpu_util


def _ctx(binding, B, N, Hq=4, Hkv=4, D=64, S_max=512, layers=1):
    return binding.VerifyContext(B, N, Hq, Hkv, D, S_max, layers)


def _mask_gpu(ctx, gu, parents):
    B, N = parents.shape
    W = (N + 63) // 64
    mask = torch.zeros((B, N, W), dtype=torch.int64, device="cuda")
    depth = torch.full((B, N), -7, dtype=torch.int32, device="cuda")
    ctx.tree_mask_build(gu.i32_dev(parents), mask, depth)
    torch.cuda.synchronize()
    return gu.u64_host(mask), depth.cpu().numpy()


@pytest.mark.parametrize("name", ["tiny", "llava7b", "qwen7b", "llava13b_b4", "qwen3b_S2048_N128_B8",
                                  "qwen3b_S2048_N16_B4", "paper_tree"])
def test_mask_matches_oracle_on_the_workload_trees(gpu, name):
    binding, gu = gpu
    cfg = synth.get_config(name)
    t = synth.make_tree_inputs(cfg)
    ctx = _ctx(binding, cfg.B, cfg.N)
    mask, depth = _mask_gpu(ctx, gu, t["parents"])
    want_mask, want_depth, ok = oracle.tree_mask(t["parents"])
    assert ok and np.array_equal(mask, want_mask) and np.array_equal(depth, want_depth)
    assert ctx.status_poll() == 0


def test_mask_all_trees_up_to_7_nodes_and_edge_sizes(gpu):
    binding, gu = gpu
    for N in range(1, 8):
        arrays = np.array([(-1,) + t for t in itertools.product(*[range(i) for i in range(1, N)])], dtype=np.int32)
        ctx = _ctx(binding, arrays.shape[0], N)
        mask, depth = _mask_gpu(ctx, gu, arrays)
        wm, wd, _ = oracle.tree_mask(arrays)
        assert np.array_equal(mask, wm) and np.array_equal(depth, wd)
    rng = np.random.Generator(np.random.Philox(3))
    for N in (63, 64, 65, 127, 128):
        parents = np.stack([synth.draw_tree(N, 40, 0, rng) for _ in range(5)] +
                           [np.arange(-1, N - 1, dtype=np.int32)])
        ctx = _ctx(binding, 6, N)
        mask, depth = _mask_gpu(ctx, gu, parents)
        wm, wd, _ = oracle.tree_mask(parents)
        assert np.array_equal(mask, wm) and np.array_equal(depth, wd)


def test_mask_bad_parents_set_status_and_do_not_fault(gpu):
    binding, gu = gpu
    parents = np.array([[-1, 0, 5, 1, 2], [-1, 0, 1, 2, 0], [0, 0, 1, 2, 3]], dtype=np.int32)
    ctx = _ctx(binding, 3, 5)
    mask, depth = _mask_gpu(ctx, gu, parents)
    wm, wd, ok = oracle.tree_mask(parents)
    assert not ok
    assert np.array_equal(mask, wm) and np.array_equal(depth, wd)
    assert ctx.status_poll() == -8 and ctx.status_poll() == 0      # read-and-clear


@pytest.mark.parametrize("name", ["tiny", "llava7b", "qwen7b", "llava13b_b4", "qwen3b_S8192_N128_B8", "paper_tree"])
def test_accept_matches_oracle_on_the_workload_trees(gpu, name):
    binding, gu = gpu
    cfg = synth.get_config(name)
    for rep in range(4):
        t = synth.make_tree_inputs(cfg, seed_offset=rep)
        ctx = _ctx(binding, cfg.B, cfg.N)
        path = torch.full((cfg.B, cfg.N), 99, dtype=torch.int32, device="cuda")
        alen = torch.zeros(cfg.B, dtype=torch.int32, device="cuda")
        bonus = torch.zeros(cfg.B, dtype=torch.int32, device="cuda")
        ctx.accept(gu.i32_dev(t["draft_ids"]), gu.i32_dev(t["target_ids"]), gu.i32_dev(t["parents"]), path, alen, bonus)
        torch.cuda.synchronize()
        wp, wl, wb = oracle.accept(t["draft_ids"], t["target_ids"], t["parents"])
        assert np.array_equal(path.cpu().numpy(), wp)
        assert np.array_equal(alen.cpu().numpy(), wl) and np.array_equal(bonus.cpu().numpy(), wb)


def test_accept_exhaustive_small_trees_and_duplicate_siblings(gpu):
    binding, gu = gpu
    rows = []
    for N in range(1, 8):
        for tail in itertools.product(*[range(i) for i in range(1, N)]):
            parents = np.array((-1,) + tail, dtype=np.int32)
            target = np.arange(100, 100 + N, dtype=np.int32)
            for pat in itertools.product([0, 1], repeat=N - 1):
                draft = np.full(N, 7, dtype=np.int32)
                for i in range(1, N):
                    if pat[i - 1]:
                        draft[i] = target[parents[i]]
                rows.append((N, parents, draft, target))
    for N in range(1, 8):
        sel = [r for r in rows if r[0] == N]
        parents = np.stack([r[1] for r in sel]); draft = np.stack([r[2] for r in sel]); target = np.stack([r[3] for r in sel])
        B = parents.shape[0]
        ctx = _ctx(binding, B, N)
        path = torch.zeros((B, N), dtype=torch.int32, device="cuda")
        alen = torch.zeros(B, dtype=torch.int32, device="cuda"); bonus = torch.zeros(B, dtype=torch.int32, device="cuda")
        ctx.accept(gu.i32_dev(draft), gu.i32_dev(target), gu.i32_dev(parents), path, alen, bonus)
        wp, wl, wb = oracle.accept(draft, target, parents)
        assert np.array_equal(path.cpu().numpy(), wp) and np.array_equal(alen.cpu().numpy(), wl)
        assert np.array_equal(bonus.cpu().numpy(), wb)
    # duplicate siblings (hand-worked): the longer branch wins
    ctx = _ctx(binding, 1, 4)
    path = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
    alen = torch.zeros(1, dtype=torch.int32, device="cuda"); bonus = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.accept(gu.i32_dev([[0, 5, 5, 9]]), gu.i32_dev([[5, 1, 9, 4]]), gu.i32_dev([[-1, 0, 0, 2]]), path, alen, bonus)
    assert path.cpu().tolist() == [[0, 2, 3, -1]] and alen.item() == 3 and bonus.item() == 4


def test_accept_bad_tree_returns_root_only(gpu):
    binding, gu = gpu
    ctx = _ctx(binding, 2, 4)
    path = torch.zeros((2, 4), dtype=torch.int32, device="cuda")
    alen = torch.zeros(2, dtype=torch.int32, device="cuda"); bonus = torch.zeros(2, dtype=torch.int32, device="cuda")
    ctx.accept(gu.i32_dev([[0, 5, 6, 7], [0, 5, 6, 7]]), gu.i32_dev([[5, 6, 7, 8], [5, 6, 7, 8]]),
               gu.i32_dev([[-1, 0, 3, 1], [-1, 0, 1, 2]]), path, alen, bonus)
    assert path.cpu().tolist() == [[0, -1, -1, -1], [0, 1, 2, 3]]
    assert alen.cpu().tolist() == [1, 4] and bonus.cpu().tolist() == [5, 8]
    assert ctx.status_poll() == -8


def _compact_case(binding, gu, B, Hkv, D, S_max, N, layers, kv_len, paths, seed=0):
    rng = np.random.default_rng(seed)
    ctx = binding.VerifyContext(B, N, Hkv, Hkv, D, S_max, layers)
    host, dev = [], []
    for l in range(layers):
        k = rng.integers(0, 65536, size=(B, Hkv, S_max, D), dtype=np.int64).astype(np.uint16)
        v = rng.integers(0, 65536, size=(B, Hkv, S_max, D), dtype=np.int64).astype(np.uint16)
        kd, vd = gu.bf16_dev(k), gu.bf16_dev(v)
        ctx.cache_register(l, kd, vd)
        host.append((k, v)); dev.append((kd, vd))
    path = np.full((B, N), -1, dtype=np.int32)
    alen = np.zeros(B, dtype=np.int32)
    for b, p in enumerate(paths):
        path[b, :len(p)] = p; alen[b] = len(p)
    out_len = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    ctx.kv_compact(0, layers, gu.i32_dev(path), gu.i32_dev(alen), gu.i32_dev(kv_len), out_len)
    torch.cuda.synchronize()
    for l in range(layers):
        wk, wv, wl = oracle.kv_compact(host[l][0], host[l][1], path, alen, kv_len)
        assert np.array_equal(gu.bf16_bits(dev[l][0]), wk), f"K differs in layer {l}"
        assert np.array_equal(gu.bf16_bits(dev[l][1]), wv), f"V differs in layer {l}"
        assert np.array_equal(out_len.cpu().numpy(), wl)
    return ctx


@pytest.mark.parametrize("D", [64, 128])
def test_compact_whole_buffer_bit_exact_with_adversarial_paths(gpu, D):
    binding, gu = gpu
    ctx = _compact_case(binding, gu, 4, 3, D, 96, 8, 3, [17, 40, 0, 88],
                        [[0, 2, 3], [0, 1, 3, 6], [0, 1, 2, 3, 4, 5, 6, 7], [0, 7]])
    assert ctx.status_poll() == 0


def test_compact_long_paths_cross_the_16_row_pass_boundary(gpu):
    binding, gu = gpu
    N = 128
    rng = np.random.default_rng(1)
    paths = []
    for L in (128, 40, 17, 16):
        p = np.sort(rng.choice(np.arange(1, N), size=L - 1, replace=False)).tolist()
        paths.append([0] + p)
    _compact_case(binding, gu, 4, 2, 128, 512, N, 2, [300, 0, 384, 77], paths)


def test_compact_workload_paths_from_acceptance(gpu):
    binding, gu = gpu
    cfg = synth.get_config("llava13b_b4")
    t = synth.make_tree_inputs(cfg)
    wp, wl, _ = oracle.accept(t["draft_ids"], t["target_ids"], t["parents"])
    paths = [wp[b, :wl[b]].tolist() for b in range(cfg.B)]
    kv_len = np.array([100, 37, 0, 250], dtype=np.int32)
    _compact_case(binding, gu, cfg.B, 5, 128, 320, cfg.N, 2, kv_len, paths)


def test_compact_out_of_range_sequence_is_skipped_with_status(gpu):
    binding, gu = gpu
    rng = np.random.default_rng(2)
    B, Hkv, D, S_max, N = 2, 2, 64, 64, 8
    ctx = binding.VerifyContext(B, N, Hkv, Hkv, D, S_max, 1)
    k = rng.integers(0, 65536, size=(B, Hkv, S_max, D), dtype=np.int64).astype(np.uint16)
    kd, vd = gu.bf16_dev(k), gu.bf16_dev(k)
    ctx.cache_register(0, kd, vd)
    path = np.array([[0, 3, -1, -1, -1, -1, -1, -1]] * 2, dtype=np.int32)
    ctx.kv_compact(0, 1, gu.i32_dev(path), gu.i32_dev([2, 2]), gu.i32_dev([60, 10]), None)   # 60 + 8 > 64
    torch.cuda.synchronize()
    got = gu.bf16_bits(kd)
    assert np.array_equal(got[0], k[0])                       # rejected sequence untouched
    wk, _, _ = oracle.kv_compact(k[1:], k[1:], path[1:], [2], [10])
    assert np.array_equal(got[1], wk[0])
    assert ctx.status_poll() == -4
    # host-side validation
    with pytest.raises(binding.VispecError):
        ctx.kv_compact(0, 2, gu.i32_dev(path), gu.i32_dev([2, 2]), gu.i32_dev([1, 1]), None)   # layer range
    kvl = gu.i32_dev([1, 1])
    with pytest.raises(binding.VispecError):
        ctx.kv_compact(0, 1, gu.i32_dev(path), gu.i32_dev([2, 2]), kvl, kvl)                   # aliasing


def _accept_commit_case(binding, gu, cfg_name, Hkv, D, layers, kv_len, S_max, seed=0):
    """vispec_accept_commit against oracle.accept followed by oracle.kv_compact, whole buffers bit-exact."""
    cfg = synth.get_config(cfg_name)
    t = synth.make_tree_inputs(cfg)
    B, N = cfg.B, cfg.N
    rng = np.random.default_rng(seed)
    ctx = binding.VerifyContext(B, N, Hkv, Hkv, D, S_max, layers)
    host, dev = [], []
    for l in range(layers):
        k = rng.integers(0, 65536, size=(B, Hkv, S_max, D), dtype=np.int64).astype(np.uint16)
        v = rng.integers(0, 65536, size=(B, Hkv, S_max, D), dtype=np.int64).astype(np.uint16)
        kd, vd = gu.bf16_dev(k), gu.bf16_dev(v)
        ctx.cache_register(l, kd, vd)
        host.append((k, v)); dev.append((kd, vd))
    path = torch.full((B, N), -9, dtype=torch.int32, device="cuda")
    alen = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    bonus = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    out_len = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    ctx.accept_commit(0, layers, gu.i32_dev(t["draft_ids"]), gu.i32_dev(t["target_ids"]), gu.i32_dev(t["parents"]),
                      gu.i32_dev(kv_len), path, alen, bonus, out_len)
    torch.cuda.synchronize()
    wp, wl, wb = oracle.accept(t["draft_ids"], t["target_ids"], t["parents"])
    assert np.array_equal(path.cpu().numpy(), wp) and np.array_equal(alen.cpu().numpy(), wl)
    assert np.array_equal(bonus.cpu().numpy(), wb)
    for l in range(layers):
        wk, wv, wn = oracle.kv_compact(host[l][0], host[l][1], wp, wl, kv_len)
        assert np.array_equal(gu.bf16_bits(dev[l][0]), wk), f"K differs in layer {l}"
        assert np.array_equal(gu.bf16_bits(dev[l][1]), wv), f"V differs in layer {l}"
        assert np.array_equal(out_len.cpu().numpy(), wn)
    assert ctx.status_poll() == 0
    assert ctx.launch_count() == 1
    return ctx


def test_accept_commit_in_one_launch_matches_accept_then_compact(gpu):
    binding, gu = gpu
    _accept_commit_case(binding, gu, "llava13b_b4", 5, 128, 3, np.array([100, 37, 0, 250], dtype=np.int32), 320)
    _accept_commit_case(binding, gu, "qwen3b_S2048_N128_B8", 2, 128, 2,
                        np.array([0, 1, 127, 128, 129, 300, 77, 5], dtype=np.int32), 512, seed=3)
    _accept_commit_case(binding, gu, "tiny", 4, 64, 1, np.array([256], dtype=np.int32), 320, seed=4)


def test_accept_commit_bad_tree_and_overlong_sequence(gpu):
    binding, gu = gpu
    rng = np.random.default_rng(5)
    B, Hkv, D, S_max, N = 2, 2, 64, 64, 4
    ctx = binding.VerifyContext(B, N, Hkv, Hkv, D, S_max, 1)
    k = rng.integers(0, 65536, size=(B, Hkv, S_max, D), dtype=np.int64).astype(np.uint16)
    kd, vd = gu.bf16_dev(k), gu.bf16_dev(k)
    ctx.cache_register(0, kd, vd)
    path = torch.zeros((B, N), dtype=torch.int32, device="cuda")
    alen = torch.zeros(B, dtype=torch.int32, device="cuda"); bonus = torch.zeros(B, dtype=torch.int32, device="cuda")
    out_len = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    # sequence 0: invalid parent link -> root only; sequence 1: 61 + 4 > 64 -> accepted path reported, nothing committed
    ctx.accept_commit(0, 1, gu.i32_dev([[0, 5, 6, 7], [0, 5, 6, 7]]), gu.i32_dev([[5, 6, 7, 8], [5, 6, 7, 8]]),
                      gu.i32_dev([[-1, 0, 3, 1], [-1, 0, 1, 2]]), gu.i32_dev([10, 61]), path, alen, bonus, out_len)
    torch.cuda.synchronize()
    assert path.cpu().tolist() == [[0, -1, -1, -1], [0, 1, 2, 3]]
    assert alen.cpu().tolist() == [1, 4] and bonus.cpu().tolist() == [5, 8]
    assert out_len.cpu().tolist() == [11, -1]
    assert np.array_equal(gu.bf16_bits(kd), k)            # root-only commit moves nothing; sequence 1 untouched
    assert ctx.status_poll() in (-8, -4)                  # the first recorded of the two
