"""Parity of the CUDA path (called through the C ABI) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import pamm_oracle as orc
from paper_2506_02939_b200 import build as pamm_build, synth

pamm_build.build()
from paper_2506_02939_b200 import pamm  # noqa: E402
from tests import parity  # noqa: E402

pytestmark = pytest.mark.gpu


def _idx(b, k, seed):
    return np.sort(np.random.default_rng(seed).choice(b, size=k, replace=False)).astype(np.int32)


# (b, n, m, k, dtype): several tiles, ragged tails in every dimension, k = 1
SMALL = [
    (300, 72, 40, 5, "f32"),
    (1000, 136, 264, 17, "bf16"),
    (4133, 512, 520, 64, "bf16"),
    (777, 2056, 1032, 128, "bf16"),
    (2500, 200, 96, 1, "bf16"),
    (1027, 516, 772, 4, "f32"),
    (640, 64, 6152, 96, "bf16"),
    (129, 8, 8, 129, "bf16"),
    (5000, 1024, 256, 256, "bf16"),
    (260, 24, 12280, 8, "bf16"),       # dY rows of 24 KiB: four 16-byte chunks per consumer thread
    (96, 16, 24584, 8, "bf16"),        # rows too wide for the shared-memory ring: column-slab path
    (500, 32, 2600, 12, "bf16"),       # dY rows of 5.2 KB: two rows per ring slot
    (333, 40, 3076, 6, "f32"),         # fp32 rows of 769 chunks: two per consumer thread
]


@pytest.mark.parametrize("b,n,m,k,dtype", SMALL)
@pytest.mark.parametrize("fused", [True, False])
def test_small_cases(b, n, m, k, dtype, fused):
    X, dY = synth.random_case(b, n, m, dtype, seed=b + k, centres=max(2, k // 2), dy_scale=1e-3)
    rep = parity.run_and_compare(X, dY, k, seed=7 + k, fused=fused)
    assert rep.unexplained == 0


def test_many_rows_ragged_everywhere():
    # more rows than 148 x 1024 (several sort blocks per SM, ranges of ~1350 rows per CTA), nothing a multiple of a tile
    X, dY = synth.random_case(200003, 264, 520, "bf16", seed=51, centres=40, dy_scale=1e-3)
    rep = parity.run_and_compare(X, dY, 96, seed=52, products=True)
    assert rep.unexplained == 0


def test_largest_generator_count_of_the_tensor_core_path():
    # k = 4096: sixteen chunks of 256 generators with a running argmax per row; k = 4097 takes the CUDA-core path
    X, dY = synth.random_case(4500, 128, 72, "bf16", seed=53, centres=300, dy_scale=1e-3)
    parity.run_and_compare(X, dY, 4096, seed=54, products=True)
    parity.run_and_compare(X[:4200], dY[:4200], 4097, seed=55)


def test_ragged_columns_with_padded_leading_dimension():
    # n and m are not multiples of the 16-byte vector; the row stride is
    X, dY = synth.random_case(700, 70, 45, "f32", seed=3, centres=6)
    parity.run_and_compare(X, dY, 9, seed=1, ldx=72, ldy=48)
    X, dY = synth.random_case(700, 67, 83, "bf16", seed=4, centres=6)
    parity.run_and_compare(X, dY, 9, seed=1, ldx=72, ldy=88)


def test_k_equals_b_reproduces_exact_product():
    X, dY = synth.random_case(384, 96, 80, "bf16", seed=5)
    rep = parity.run_and_compare(X, dY, 384, idx_in=np.arange(384, dtype=np.int32))
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    idx, C, invn, f, alpha = pamm.compress_fused(Xd, 384, 0, idx_in=torch.arange(384, dtype=torch.int32, device="cuda"))
    assert torch.equal(f.cpu(), torch.arange(384, dtype=torch.int32))
    assert torch.allclose(alpha, torch.ones_like(alpha), rtol=1e-6, atol=0)
    dW = pamm.contract_weight_grad(C, f, alpha, dYd).cpu().numpy()
    exact = synth.to_f64(X).T @ synth.to_f64(dY)
    assert parity.rel_fro(dW, exact) <= 1e-2
    assert parity.rel_fro(dW, exact) <= 1e-4      # in fact only fp32 rounding remains


def test_rank_one_input_reproduces_exact_product():
    rng = np.random.default_rng(6)
    u = (rng.integers(1, 9, size=512) * rng.choice([-1, 1], size=512)).astype(np.float32)
    v = rng.integers(-8, 9, size=64).astype(np.float32)
    v[0] = 5
    X = np.outer(u, v).astype(np.float32)
    _, dY = synth.random_case(512, 64, 48, "f32", seed=7)
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    idx, C, invn, f, alpha = pamm.compress_fused(Xd, 3, 11)
    dW = pamm.contract_weight_grad(C, f, alpha, dYd).cpu().numpy()
    exact = X.astype(np.float64).T @ dY.astype(np.float64)
    assert parity.rel_fro(dW, exact) <= 1e-5
    # every generator ties on every row: whatever f the GPU picked, the oracle calls it a near-tie
    rep = parity.run_and_compare(X, dY, 3, seed=11)
    assert rep.unexplained == 0 and rep.explained_by_rounding == 0


def test_padding_rows_share_f_and_alpha_and_zero_rows():
    inp = synth.make_inputs("c2", num_seqs=16)
    X, dY = inp.X, inp.dY
    k = 8
    parity.run_and_compare(X, dY, k, seed=3)
    # force a zero generator and a duplicated generator row through caller-chosen indices
    pads = inp.pad_rows
    zero_rows = pads[np.all((X[pads] & 0x7FFF) == 0, axis=1)]
    dup_rows = pads[~np.all((X[pads] & 0x7FFF) == 0, axis=1)]
    assert len(zero_rows) > 2 and len(dup_rows) > 2
    idx = np.array([5, dup_rows[0], 900, zero_rows[0], dup_rows[1], 2000], np.int32)
    rep = parity.run_and_compare(X, dY, len(idx), idx_in=idx)
    Xd = parity.to_device(X)
    _, C, invn, f, alpha = pamm.compress_fused(Xd, len(idx), 0, idx_in=torch.from_numpy(idx).cuda())
    f, alpha = f.cpu().numpy(), alpha.cpu().numpy()
    assert np.all(f[dup_rows] == 1) and np.all(alpha[dup_rows] == alpha[dup_rows[0]])   # lowest of the twins
    assert abs(alpha[dup_rows[0]] - 1.0) < 1e-6
    assert np.all(f[zero_rows] == 0) and np.all(alpha[zero_rows] == 0.0)
    assert not np.any(f == 3) and np.all(np.isfinite(alpha))


def test_results_are_bit_reproducible():
    X, dY = synth.random_case(3000, 256, 520, "bf16", seed=8, centres=20)
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    outs = []
    for _ in range(3):
        idx, C, invn, f, alpha = pamm.compress_fused(Xd, 48, 5)
        Bt = torch.empty((48, 520), dtype=torch.float32, device="cuda")
        dW = pamm.contract_weight_grad(C, f, alpha, dYd, Btilde=Bt)
        outs.append([t.clone() for t in (idx, C, invn, f, alpha, Bt, dW)])
    for o in outs[1:]:
        for a, b_ in zip(outs[0], o):
            assert torch.equal(a.view(torch.uint8) if a.dtype == torch.bfloat16 else a,
                               b_.view(torch.uint8) if b_.dtype == torch.bfloat16 else b_)


@pytest.mark.parametrize("b,n,m,k", [(1500, 136, 264, 24), (1300, 200, 392, 200), (2100, 72, 3080, 300)])
def test_outputs_stay_inside_their_buffers(b, n, m, k):
    # guard regions around every output and the workspace: k <= 128 and k > 128 products, one and two rows per ring slot
    X, dY = synth.random_case(b, n, m, "bf16", seed=9, centres=10)
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    G = 64

    def guarded(shape, dtype):
        numel = int(np.prod(shape))
        raw = torch.full((numel + 2 * G,), -7, dtype=dtype, device="cuda") if dtype != torch.bfloat16 else \
            torch.full((numel + 2 * G,), -7.0, dtype=dtype, device="cuda")
        return raw, raw[G:G + numel].view(shape)

    raws = {}
    raws["idx"], idx = guarded((k,), torch.int32)
    raws["C"], C = guarded((k, n), torch.bfloat16)
    raws["invn"], invn = guarded((2 * k,), torch.float32)
    raws["f"], f = guarded((b,), torch.int32)
    raws["alpha"], alpha = guarded((b,), torch.float32)
    raws["Bt"], Bt = guarded((k, m), torch.float32)
    raws["dW"], dW = guarded((n, m), torch.float32)
    need = pamm.workspace_bytes(pamm.WS_CONTRACT, b, n, m, k, pamm.BF16)
    ws_raw = torch.full((need + 512,), 0x5A, dtype=torch.uint8, device="cuda")
    ws = ws_raw[256:256 + need]
    pamm.compress_fused(Xd, k, 2, idx_out=idx, C=C, c_invnorm=invn, f=f, alpha=alpha)
    pamm.contract_weight_grad(C, f, alpha, dYd, Btilde=Bt, dW=dW, workspace=ws)
    assert pamm.last_device_status() == pamm.OK
    for name, raw in raws.items():
        head, tail = raw[:G].float().cpu(), raw[-G:].float().cpu()
        assert torch.all(head == -7) and torch.all(tail == -7), name
    assert torch.all(ws_raw[:256] == 0x5A) and torch.all(ws_raw[-256:] == 0x5A)
    assert torch.all(torch.isfinite(dW))


def test_device_side_problems_raise_a_status_not_a_fault():
    X, dY = synth.random_case(256, 64, 32, "f32", seed=10)
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    assert pamm.last_device_status() == pamm.OK
    bad = torch.tensor([3, 999, 7, 7], dtype=torch.int32, device="cuda")     # out of range + duplicate
    idx, C, invn = pamm.select_generators(Xd, 4, idx_in=bad)
    assert pamm.last_device_status() == pamm.ERR_BAD_INDEX
    assert pamm.last_device_status() == pamm.OK                               # reading clears it
    assert idx.cpu().tolist() == [3, 255, 7, 7]
    f = torch.zeros(256, dtype=torch.int32, device="cuda")
    f[10] = 4
    f[11] = -1
    alpha = torch.ones(256, dtype=torch.float32, device="cuda")
    Bt = pamm.contract(f, alpha, dYd, 4)
    assert pamm.last_device_status() == pamm.ERR_BAD_INDEX
    keep = np.ones(256, bool)
    keep[[10, 11]] = False
    assert np.allclose(Bt[0].cpu().numpy(), dY[keep].astype(np.float64).sum(axis=0), rtol=1e-4, atol=1e-6)
    assert torch.all(Bt[1:] == 0)


def test_few_generators_take_the_three_launch_path():
    # k <= 8: selection + compression in one launch, contraction without a sort, reduction + product in one launch
    X, dY = synth.random_case(3000, 200, 392, "bf16", seed=19, centres=6, dy_scale=1e-3)
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    n0 = pamm.launch_count()
    idx, C, invn, f, alpha = pamm.compress_fused(Xd, 6, 3)
    Bt = pamm.alloc_matrix(6, 392, torch.float32)
    dW = pamm.contract_weight_grad(C, f, alpha, dYd, Btilde=Bt)
    assert pamm.launch_count() - n0 == 3
    # the same selection and the same assignment as the general kernels give
    idx2, C2, invn2 = pamm.select_generators(Xd, 6, 3)
    f2, alpha2 = pamm.compress(Xd, C2, invn2)
    assert torch.equal(idx, idx2) and torch.equal(C.view(torch.int16), C2.view(torch.int16))
    assert torch.allclose(invn, invn2, rtol=1e-6, atol=0) and torch.equal(f, f2)
    assert torch.allclose(alpha, alpha2, rtol=1e-5, atol=1e-7)
    # caller's indices that are out of range or repeated: clamped, kept, reported -- as the selection kernel does
    bad = torch.tensor([3, 99999, 7, 7], dtype=torch.int32, device="cuda")
    idx, *_ = pamm.compress_fused(Xd, 4, idx_in=bad)
    assert pamm.last_device_status() == pamm.ERR_BAD_INDEX
    assert idx.cpu().tolist() == [3, 2999, 7, 7]
    # an assignment outside [0, k) is skipped and reported by the sort-free contraction too
    f[10] = 6
    Bt_bad = pamm.alloc_matrix(6, 392, torch.float32)
    pamm.contract_weight_grad(C, f, alpha, dYd, Btilde=Bt_bad)
    assert pamm.last_device_status() == pamm.ERR_BAD_INDEX
    keep = np.ones(3000, bool)
    keep[10] = False
    ref = orc.contract(np.where(keep, f.cpu().numpy(), 0).astype(np.int32), np.where(keep, alpha.cpu().numpy(), 0.0), dY, 6)
    assert parity.rel_fro(Bt_bad.cpu().numpy(), ref) <= 1e-5


def test_unfused_stage_inputs_from_elsewhere():
    # contract / weight_grad accept any (f, alpha, B~), not only what compress produced
    rng = np.random.default_rng(12)
    b, m, k, n = 2000, 300, 10, 40
    _, dY = synth.random_case(b, 8, m, "bf16", seed=13)
    f = rng.integers(0, k, size=b).astype(np.int32)
    f[f == 4] = 5                                                     # an empty segment
    a = rng.standard_normal(b).astype(np.float32)
    Bt = pamm.contract(torch.from_numpy(f).cuda(), torch.from_numpy(a).cuda(), parity.to_device(dY, ld=304), k)
    ref = orc.contract(f, a.astype(np.float64), dY, k)
    assert parity.rel_fro(Bt.cpu().numpy(), ref) <= 1e-5
    assert torch.all(Bt[4] == 0)
    Cb, _ = synth.random_case(k, n, 8, "bf16", seed=14)
    dW = pamm.weight_grad(parity.to_device(Cb), Bt)
    ref = orc.weight_grad(synth.to_f64(Cb), Bt.cpu().numpy().astype(np.float64))
    assert parity.rel_fro(dW.cpu().numpy(), ref) <= 1e-4


def test_host_buffer_step_matches_device_path():
    X, dY = synth.random_case(1200, 128, 200, "bf16", seed=15, centres=12, dy_scale=1e-3)
    Xh = torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).pin_memory()
    dYh = torch.from_numpy(dY.view(np.int16)).view(torch.bfloat16).pin_memory()
    dWh = torch.empty((128, 200), dtype=torch.float32).pin_memory()
    fh = torch.empty(1200, dtype=torch.int32).pin_memory()
    ah = torch.empty(1200, dtype=torch.float32).pin_memory()
    arena = pamm.alloc_workspace(pamm.WS_STEP_HOST, 1200, 128, 200, 16, pamm.BF16)
    pamm.qkv_step_host(Xh, dYh, 16, 21, dWh, arena, f_host=fh, alpha_host=ah)
    assert pamm.last_device_status() == pamm.OK
    idx, C, invn, f, alpha = pamm.compress_fused(Xh.cuda(), 16, 21)
    dW = pamm.contract_weight_grad(C, f, alpha, dYh.cuda())
    assert torch.equal(fh, f.cpu()) and torch.equal(ah, alpha.cpu()) and torch.equal(dWh, dW.cpu())


# ---- the five workloads at full size, in the launch configuration the benchmark times ----

@pytest.mark.parametrize("name", ["c1", "c2", "c4", "c5"])
def test_workload_full_size(name):
    inp = synth.make_inputs(name)
    w = inp.workload
    rep = parity.run_and_compare(inp.X, inp.dY, w.ks[0], seed=w.index_seed, products=True)
    parity.record(f"{name} k={w.ks[0]}", rep)


def test_workload_c3_ratio_sweep():
    inp = synth.make_inputs("c3")
    w = inp.workload
    for k in w.ks:
        rep = parity.run_and_compare(inp.X, inp.dY, k, seed=w.index_seed, products=True)
        parity.record(f"c3 k={k}", rep)


def test_layer_stack_keeps_only_the_compressed_state():
    """c5-shaped layers at reduced batch: forward of every layer first (X is not needed afterwards),
    backward in reverse order from the kept (C, f, alpha) only; the bytes kept follow k n e + 8 b."""
    L = 3
    layers = [synth.make_inputs("c5", num_seqs=1, seed=4 + 100 * l) for l in range(L)]
    w = layers[0].workload
    b, n, m, k = layers[0].b, w.n, w.m, w.ks[0]
    kept = []
    for l, inp in enumerate(layers):
        Xd = parity.to_device(inp.X)
        idx, C, invn, f, alpha = pamm.compress_fused(Xd, k, w.index_seed + 100 * l)
        kept.append((idx, C, f, alpha))
        del Xd                                                     # the layer's input is gone after its forward pass
    kept_bytes = sum(C.numel() * 2 + f.numel() * 4 + alpha.numel() * 4 for _, C, f, alpha in kept)
    assert kept_bytes == L * (k * n * 2 + 8 * b)
    assert pamm.saved_bytes(b, n, k, pamm.BF16)["pamm"] * L == kept_bytes
    assert L * b * n * 2 / kept_bytes > 100                        # 341x at the full batch, 114x at this one
    rng = np.random.default_rng(0)
    rr, cc = rng.integers(0, n, 2048), rng.integers(0, m, 2048)
    for l in reversed(range(L)):
        idx, C, f, alpha = kept[l]
        dW = pamm.contract_weight_grad(C, f, alpha, parity.to_device(layers[l].dY)).cpu().numpy()
        assert pamm.last_device_status() == pamm.OK
        C64 = synth.to_f64(parity.from_device_bits(C))
        Bt = orc.contract(f.cpu().numpy(), alpha.cpu().numpy().astype(np.float64), layers[l].dY, k)
        ref = np.einsum("js,js->s", C64[:, rr], Bt[:, cc])
        assert parity.rel_fro(dW[rr, cc], ref) <= 1e-2


@pytest.mark.parametrize("layout", [pamm.DW_NM, pamm.DW_MN])
@pytest.mark.parametrize("k,n,m,dtype", [(24, 136, 264, "bf16"), (200, 72, 136, "bf16"), (5, 40, 52, "f32")])
def test_weight_grad_accumulate_adds_to_dW(k, n, m, dtype, layout):
    # the three product kernels (persistent tcgen05, chunked tcgen05, CUDA cores): dW += C^T B~, twice, either layout
    Cb, _ = synth.random_case(k, n, 8, dtype, seed=21)
    Bt = torch.from_numpy(np.random.default_rng(22).standard_normal((k, m)).astype(np.float32)).cuda()
    C = parity.to_device(Cb)
    shape = (n, m) if layout == pamm.DW_NM else (m, n)
    base = torch.from_numpy(np.random.default_rng(23).standard_normal(shape).astype(np.float32)).cuda()
    once = pamm.weight_grad(C, Bt, layout=layout)
    assert once.shape == shape
    dW = base.clone()
    pamm.weight_grad_accumulate(C, Bt, dW, layout=layout)
    assert torch.allclose(dW, base + once, rtol=1e-6, atol=1e-6)
    pamm.weight_grad_accumulate(C, Bt, dW, layout=layout)
    assert torch.allclose(dW, base + 2 * once, rtol=1e-6, atol=1e-5)
    assert pamm.last_device_status() == pamm.OK


# ---- storage options of the outputs: dW in fp32 / bf16, n x m / m x n; f in 32 / 16 / 8 bits ----

@pytest.mark.parametrize("layout", [pamm.DW_NM, pamm.DW_MN])
@pytest.mark.parametrize("dw_dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("b,n,m,k,dtype", [
    (1500, 264, 392, 48, "bf16"),      # persistent tcgen05 product (k <= 128), ragged tiles in both directions
    (1200, 136, 200, 200, "bf16"),     # chunked tcgen05 product (k > 128)
    (900, 72, 100, 5, "f32"),          # CUDA-core product
    (700, 40, 56, 6, "bf16"),          # bf16 generators with k < 8: CUDA-core product
])
def test_weight_gradient_types_and_layouts(b, n, m, k, dtype, dw_dtype, layout):
    X, dY = synth.random_case(b, n, m, dtype, seed=31 + k, centres=max(2, k // 2), dy_scale=1e-3)
    rep = parity.run_and_compare(X, dY, k, seed=3 + k, dw_dtype=dw_dtype, layout=layout)
    assert rep.unexplained == 0


def test_fp32_weight_gradient_in_the_papers_layout_is_unchanged_by_the_options():
    # the transposed layout holds the same numbers; the bf16 one their nearest-even roundings
    X, dY = synth.random_case(2000, 264, 392, "bf16", seed=41, centres=12, dy_scale=1e-3)
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    for k in (48, 200):
        idx, C, invn, f, alpha = pamm.compress_fused(Xd, k, 5)
        Bt = pamm.contract(f, alpha, dYd, k)
        ref = pamm.weight_grad(C, Bt)
        assert torch.equal(pamm.weight_grad(C, Bt, layout=pamm.DW_MN).t(), ref)
        assert torch.equal(pamm.weight_grad(C, Bt, dw_dtype=torch.bfloat16), ref.to(torch.bfloat16))
        assert torch.equal(pamm.weight_grad(C, Bt, dw_dtype=torch.bfloat16, layout=pamm.DW_MN).t(), ref.to(torch.bfloat16))
    assert pamm.last_device_status() == pamm.OK


@pytest.mark.parametrize("f_dtype,b,n,m,k,dtype", [
    (torch.uint8, 3000, 136, 264, 200, "bf16"),
    (torch.uint8, 1000, 72, 40, 256, "bf16"),         # the largest k a byte can name
    (torch.int16, 2500, 200, 136, 700, "bf16"),       # unsigned 16-bit entries (torch's int16 as storage)
    (torch.uint8, 800, 64, 48, 3, "f32"),             # CUDA-core compress
])
def test_narrow_assignment_storage(f_dtype, b, n, m, k, dtype):
    X, dY = synth.random_case(b, n, m, dtype, seed=17 + k, centres=max(2, k // 2), dy_scale=1e-3)
    for fused in (True, False):
        rep = parity.run_and_compare(X, dY, k, seed=2 + k, f_dtype=f_dtype, fused=fused, products=fused)
        assert rep.unexplained == 0
    # and the same bits as the 32-bit path
    Xd = parity.to_device(X)
    _, C, invn, f32, a32 = pamm.compress_fused(Xd, k, 9)
    _, _, _, fn, an = pamm.compress_fused(Xd, k, 9, f_dtype=f_dtype)
    wide = fn.to(torch.int32) & (0xFFFF if f_dtype == torch.int16 else 0xFF)
    assert torch.equal(wide, f32) and torch.equal(an, a32)
    with pytest.raises(pamm.PammError):
        pamm.compress_fused(Xd, 257, 9, f_dtype=torch.uint8)


# ---- the counts of f that the forward pass leaves for the backward pass ----

@pytest.mark.parametrize("b,n,m,k,dtype", [(5000, 136, 264, 40, "bf16"), (3000, 64, 72, 900, "bf16"), (2048, 72, 96, 12, "f32")])
def test_sort_products_of_the_forward_pass(b, n, m, k, dtype):
    # tensor-core compress, the three-launch sort (many generators), CUDA-core compress
    X, dY = synth.random_case(b, n, m, dtype, seed=61, centres=max(2, k // 3), dy_scale=1e-3)
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    code = pamm.BF16 if dtype == "bf16" else pamm.F32
    sp = pamm.alloc_workspace(pamm.WS_COMPRESS, b, n, m, k, code)
    idx, C, invn, f, alpha = pamm.compress_fused(Xd, k, 4, sort_products=sp)
    # the products are histograms of f per block of rows (equal blocks, at most one per SM, a multiple of 64 rows):
    # their column sums are the histogram of the whole f
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    rows_per_block = max(64, (-(-b // sms) + 63) // 64 * 64)
    nblk = -(-b // rows_per_block)
    counts = sp[: nblk * k * 4].view(torch.int32).view(nblk, k).to(torch.int64)
    assert torch.equal(counts.sum(dim=0), torch.bincount(f.to(torch.int64), minlength=k))
    assert torch.equal(counts[0], torch.bincount(f[:rows_per_block].to(torch.int64), minlength=k))
    launches0 = pamm.launch_count()
    with_products = pamm.contract(f, alpha, dYd, k, sort_products=sp)
    n_with = pamm.launch_count() - launches0
    launches0 = pamm.launch_count()
    without = pamm.contract(f, alpha, dYd, k)
    n_without = pamm.launch_count() - launches0
    assert n_with == n_without - 1                                   # the counting launch is gone
    assert torch.equal(with_products, without)
    assert pamm.last_device_status() == pamm.OK


def test_sort_products_of_another_assignment_are_reported_not_trusted():
    X, dY = synth.random_case(4000, 72, 136, "bf16", seed=62, centres=9, dy_scale=1e-3)
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    k = 24
    sp = pamm.alloc_workspace(pamm.WS_COMPRESS, 4000, 72, 136, k, pamm.BF16)
    idx, C, invn, f, alpha = pamm.compress_fused(Xd, k, 4, sort_products=sp)
    sp.view(torch.int32)[: 6 * k] += 1000                            # counts that do not belong to f any more
    Bt = pamm.contract(f, alpha, dYd, k, sort_products=sp)
    assert pamm.last_device_status() == pamm.ERR_BAD_INDEX           # noticed on the device, nothing faulted
    assert pamm.last_device_status() == pamm.OK
    good = pamm.contract(f, alpha, dYd, k)                           # and the library carries on
    ref = orc.contract(f.cpu().numpy(), alpha.cpu().numpy().astype(np.float64), dY, k)
    assert parity.rel_fro(good.cpu().numpy(), ref) <= 1e-5


# ---- one compression per projection, in one pass over X (Section 4) ----

@pytest.mark.parametrize("b,n,k,dtype,sets", [(3000, 264, 40, "bf16", 3), (2000, 136, 300, "bf16", 3), (1500, 72, 5, "f32", 3),
                                              (1000, 64, 100, "bf16", 2)])
def test_one_compression_per_projection(b, n, k, dtype, sets):
    ms = [136, 72, 40][:sets]
    m = sum(ms)
    X, dY = synth.random_case(b, n, m, dtype, seed=71 + k, centres=max(3, k // 2), dy_scale=1e-3)
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    tdt = Xd.dtype
    C = pamm.alloc_matrix(sets * k, n, tdt)
    invn = torch.empty(sets * 2 * k, dtype=torch.float32, device="cuda")
    idx = torch.empty(sets * k, dtype=torch.int32, device="cuda")
    for s in range(sets):                                            # an index seed per projection
        pamm.select_generators(Xd, k, seed=100 + s, idx_out=idx[s * k:(s + 1) * k], C=C[s * k:(s + 1) * k],
                               c_invnorm=invn[s * 2 * k:(s + 1) * 2 * k])
    f, alpha = pamm.compress_projections(Xd, C, invn, sets)
    assert f.shape == (sets, b) and alpha.shape == (sets, b)
    dW = pamm.alloc_matrix(n, m, torch.float32)
    col = 0
    for s in range(sets):
        # every set's result is what a compression of its own gives, bit for bit
        f1, a1 = pamm.compress(Xd, C[s * k:(s + 1) * k], invn[s * 2 * k:(s + 1) * 2 * k])
        assert torch.equal(f[s], f1) and torch.equal(alpha[s], a1)
        # the oracle, run per projection with that projection's index set
        rep = parity.Report(b=b, k=k)
        C64, q = orc.gather(X, idx[s * k:(s + 1) * k].cpu().numpy())
        f_e, a_e = parity.check_compress(X, C64, q, f[s].cpu().numpy(), alpha[s].cpu().numpy(), rep, dtype)
        # backward per projection on its own columns of dY and dW
        dYs = dYd[:, col:col + ms[s]]
        Bt = pamm.contract(f[s], alpha[s], dYs, k)
        pamm.weight_grad(C[s * k:(s + 1) * k], Bt, dW=dW[:, col:col + ms[s]])
        ref = orc.weight_grad(C64, orc.contract(f_e, a_e, np.ascontiguousarray(dY[:, col:col + ms[s]]), k))
        assert parity.rel_fro(dW[:, col:col + ms[s]].cpu().numpy(), ref) <= parity.TOL_TIGHT[dtype]
        col += ms[s]
    assert pamm.last_device_status() == pamm.OK


def test_adapter_shaped_layer_with_a_narrow_output():
    # the input of a low-rank adapter's first matrix (Section 4.7 applies the method there): m is the adapter's rank
    X, dY = synth.random_case(4096, 1288, 16, "bf16", seed=81, centres=30, dy_scale=1e-3)
    rep = parity.run_and_compare(X, dY, 32, seed=82, products=True)
    assert rep.unexplained == 0
    rep = parity.run_and_compare(X, dY, 32, seed=82, dw_dtype=torch.bfloat16, layout=pamm.DW_MN)
    assert rep.unexplained == 0


def test_contract_with_many_generators_uses_large_shared_histograms():
    # k = 13000: the per-block histograms of the sort need more than the default 48 KiB of shared memory
    rng = np.random.default_rng(61)
    b, m, k = 20000, 72, 13000
    _, dY = synth.random_case(b, 8, m, "bf16", seed=62)
    f = rng.integers(0, k, size=b).astype(np.int32)
    a = rng.standard_normal(b).astype(np.float32)
    Bt = pamm.contract(torch.from_numpy(f).cuda(), torch.from_numpy(a).cuda(), parity.to_device(dY), k)
    assert pamm.last_device_status() == pamm.OK
    ref = orc.contract(f, a.astype(np.float64), dY, k)
    assert parity.rel_fro(Bt.cpu().numpy(), ref) <= 1e-5


def test_a_wait_that_runs_out_reports_a_timeout_and_the_context_lives_on():
    assert pamm.last_device_status() == pamm.OK
    pamm.selftest_bounded_wait()                                   # waits on a barrier nothing completes, with a limit
    assert pamm.last_device_status() == pamm.ERR_TIMEOUT
    assert pamm.last_device_status() == pamm.OK
    X, dY = synth.random_case(600, 72, 40, "bf16", seed=71, centres=5, dy_scale=1e-3)
    parity.run_and_compare(X, dY, 20, seed=72)                     # the library still works afterwards


def test_a_whole_step_can_be_captured_in_a_cuda_graph():
    # launch-bound sizes profit from replaying the seven launches of a step as one graph
    X, dY = synth.random_case(2048, 512, 1536, "f32", seed=81, centres=16, dy_scale=1e-3)
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    k = 4
    idx, C, invn, f, alpha = pamm.compress_fused(Xd, k, 3)
    Bt = pamm.alloc_matrix(k, 1536, torch.float32)
    dW = pamm.alloc_matrix(512, 1536, torch.float32)
    ws = pamm.alloc_workspace(pamm.WS_CONTRACT, 2048, 512, 1536, k, pamm.F32)

    def step(stream=None):
        pamm.compress_fused(Xd, k, 3, idx_out=idx, C=C, c_invnorm=invn, f=f, alpha=alpha, stream=stream)
        pamm.contract_weight_grad(C, f, alpha, dYd, Btilde=Bt, dW=dW, workspace=ws, stream=stream)

    step()
    torch.cuda.synchronize()
    want = [t.clone() for t in (f, alpha, Bt, dW)]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step(torch.cuda.current_stream())
    for t in (f, alpha, Bt, dW):
        t.zero_()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert pamm.last_device_status() == pamm.OK
    for got, ref in zip((f, alpha, Bt, dW), want):
        assert torch.equal(got, ref)


def test_a_bf16_layer_with_many_generators_can_be_captured_in_a_cuda_graph():
    # the kernels on pairs of CTAs (cluster launches) and the product over the bf16 planes, inside a graph
    b, n, m, k = 2048, 512, 768, 256
    X, dY = synth.random_case(b, n, m, "bf16", seed=82, centres=64, dy_scale=1e-3)
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    W = parity.to_device(synth.f32_to_bf16_bits(np.random.default_rng(3).standard_normal((n, m)).astype(np.float32) / 16))
    sp = pamm.alloc_workspace(pamm.WS_COMPRESS, b, n, m, k, pamm.BF16)
    Z, idx, C, invn, f, alpha = pamm.linear_forward(Xd, W, k, 5, sort_products=sp)
    Bt = pamm.alloc_matrix(k, m, torch.float32)
    dW = pamm.alloc_matrix(n, m, torch.float32)
    dX = pamm.alloc_matrix(b, n, torch.bfloat16)
    ws = pamm.alloc_workspace(pamm.WS_CONTRACT, b, n, m, k, pamm.BF16)

    def step(stream=None):
        pamm.linear_forward(Xd, W, k, 5, Z=Z, idx_out=idx, C=C, c_invnorm=invn, f=f, alpha=alpha, sort_products=sp, stream=stream)
        pamm.contract_weight_grad(C, f, alpha, dYd, Btilde=Bt, dW=dW, sort_products=sp, workspace=ws, stream=stream)
        pamm.linear_backward_input(dYd, W, dX=dX, stream=stream)

    step()
    torch.cuda.synchronize()
    outs = (Z.view(torch.int16), f, alpha, Bt, dW, dX.view(torch.int16))
    want = [t.clone() for t in outs]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step(torch.cuda.current_stream())
    for t in outs:
        t.zero_()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert pamm.last_device_status() == pamm.OK
    for got, ref in zip(outs, want):
        assert torch.equal(got, ref)


def test_read_probes_visit_every_row_once():
    # no arithmetic of the method: the checksums only show that the probes read what they are timed for
    g = torch.Generator(device="cuda").manual_seed(5)
    data = torch.randint(-2**31, 2**31 - 1, (3001, 776), dtype=torch.int32, device="cuda", generator=g)[:, :772]   # padded rows
    words = data.to(torch.int64)
    s = pamm.probe_read(pamm.PROBE_SUM, data)
    assert (int(s.item()) - int(words.sum().item())) % 2**32 == 0
    first = int(words[:, 0].sum().item())
    s = pamm.probe_read(pamm.PROBE_ROWS, data)
    assert (int(s.item()) - first) % 2**32 == 0
    order = torch.randperm(3001, device="cuda", generator=g).to(torch.int32)
    s = pamm.probe_read(pamm.PROBE_ROWS, data, order=order)
    assert (int(s.item()) - first) % 2**32 == 0
    twice = torch.zeros(3001, dtype=torch.int32, device="cuda")          # every position reads row 0
    s = pamm.probe_read(pamm.PROBE_ROWS, data, order=twice)
    assert (int(s.item()) - 3001 * int(words[0, 0].item())) % 2**32 == 0
    assert pamm.last_device_status() == pamm.OK
    bad = order.clone()
    bad[17] = 3001
    pamm.probe_read(pamm.PROBE_ROWS, data, order=bad)
    assert pamm.last_device_status() == pamm.ERR_BAD_INDEX


def test_calls_from_a_thread_that_has_not_touched_cuda_yet():
    # a framework's worker thread (autograd's, a data loader's) may make its first CUDA call inside the library,
    # and that call may start with a tensor-map encoding, which needs a current context
    import threading
    X, dY = synth.random_case(512, 256, 384, "bf16", seed=77)
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    idx, C, invn, f, alpha = pamm.compress_fused(Xd, 32, 3)
    Bt = pamm.contract(f, alpha, dYd, 32)
    dW_main = pamm.weight_grad(C, Bt)
    dX_main = pamm.linear_backward_input(dYd, parity.to_device(synth.f32_to_bf16_bits(np.ones((256, 384), np.float32))))
    Wd = parity.to_device(synth.f32_to_bf16_bits(np.ones((256, 384), np.float32)))
    dW_thr = torch.empty_like(dW_main)
    dX_thr = torch.empty_like(dX_main)
    torch.cuda.synchronize()
    errors = []
    stream = torch.cuda.current_stream()

    def work():
        try:
            pamm.weight_grad(C, Bt, dW=dW_thr, stream=stream)
            pamm.linear_backward_input(dYd, Wd, dX=dX_thr, stream=stream)
        except Exception as e:      # noqa: BLE001
            errors.append(e)

    t = threading.Thread(target=work)
    t.start()
    t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    assert torch.equal(dW_thr, dW_main) and torch.equal(dX_thr.view(torch.int16), dX_main.view(torch.int16))
    assert pamm.last_device_status() == pamm.OK


def test_rows_with_zero_alpha_are_never_read():
    # a row with alpha = 0 adds nothing to B~ (Section 3.2: B~_j is a sum of alpha_i B_i): the backward pass leaves it
    # out of its sorted order, so whatever its row of dY holds -- here NaNs -- does not reach B~ or dW
    b, n, m, k = 3000, 256, 520, 32
    X, dY = synth.random_case(b, n, m, "bf16", seed=91, centres=20)
    zero_rows = np.arange(7, b, 13)
    X = X.copy()
    X[zero_rows] = 0                                  # all-zero rows: S = 0, alpha = 0
    poisoned = dY.copy()
    poisoned[zero_rows] = 0x7FC0                      # bf16 NaN
    cleaned = dY.copy()
    cleaned[zero_rows] = 0
    Xd = parity.to_device(X)
    for with_products in (True, False):
        sp = pamm.alloc_workspace(pamm.WS_COMPRESS, b, n, m, k, pamm.BF16) if with_products else None
        idx, C, invn, f, alpha = pamm.compress_fused(Xd, k, 4, sort_products=sp)
        assert torch.all(alpha[torch.from_numpy(zero_rows).cuda()] == 0)
        Bt_p = pamm.alloc_matrix(k, m, torch.float32)
        Bt_c = pamm.alloc_matrix(k, m, torch.float32)
        dW_p = pamm.contract_weight_grad(C, f, alpha, parity.to_device(poisoned), Btilde=Bt_p, sort_products=sp)
        dW_c = pamm.contract_weight_grad(C, f, alpha, parity.to_device(cleaned), Btilde=Bt_c, sort_products=sp)
        assert pamm.last_device_status() == pamm.OK
        assert torch.isfinite(Bt_p).all() and torch.isfinite(dW_p).all()
        assert torch.equal(Bt_p, Bt_c) and torch.equal(dW_p, dW_c)
    # and against the oracle on the cleaned input
    for products in (False, True):
        parity.run_and_compare(X, cleaned, k, seed=4, products=products)
    # a handful of generators (the path without a sort): the same rule
    idx, C, invn, f, alpha = pamm.compress_fused(Xd, 4, 4)
    dW_p = pamm.contract_weight_grad(C, f, alpha, parity.to_device(poisoned))
    dW_c = pamm.contract_weight_grad(C, f, alpha, parity.to_device(cleaned))
    assert torch.isfinite(dW_p).all() and torch.equal(dW_p, dW_c)
