"""The forward pass with the compression fused into it (Algorithm 2: Z = X W and Compress(X) in one kernel),
called through the C ABI and compared with the oracle: Z element by element, f and alpha through the same
checks as the stand-alone compression, and bit for bit against it."""
import numpy as np
import pytest
import torch

from oracle import pamm_oracle as orc
from paper_2506_02939_b200 import build as pamm_build, synth

pamm_build.build()
from paper_2506_02939_b200 import pamm  # noqa: E402
from tests import parity  # noqa: E402

pytestmark = pytest.mark.gpu


def make_weight(n, m, seed):
    rng = np.random.default_rng([seed, 5])
    return synth.f32_to_bf16_bits((rng.standard_normal((n, m), dtype=np.float32) / np.float32(np.sqrt(n))))


def z_bound(X, W, Z_ref, rows=None):
    """Z is an n-term fp32 sum rounded once to bf16: half a unit in the last place of the result (2^-9 relative,
    2^-8 allowed) plus the accumulation's n 2^-24 times the sum of the absolute values of the terms."""
    S = orc.linear_forward(parity.abs_bits(X), parity.abs_bits(W), rows=rows)
    n = X.shape[1]
    return 2.0 ** -8 * np.abs(Z_ref) + parity.SAFETY * (n + 2) * parity.U32 * S


def check_forward(X, W, k, seed, rows=None, ldx=None):
    b, n = X.shape
    m = W.shape[1]
    Xd, Wd = parity.to_device(X, ldx), parity.to_device(W)
    sp = pamm.alloc_workspace(pamm.WS_COMPRESS, b, n, m, k, pamm.BF16)
    Z, idx, C, invn, f, alpha = pamm.linear_forward(Xd, Wd, k, seed, sort_products=sp)
    assert pamm.last_device_status() == pamm.OK
    # ---- the compression: against the oracle, and bit for bit what the stand-alone entry gives ----
    rep = parity.Report(b=b, k=k)
    C64, q = parity.check_select(X, idx.cpu().numpy(), parity.from_device_bits(C), invn.cpu().numpy().astype(np.float64), k, None, seed)
    parity.check_compress(X, C64, q, f.cpu().numpy(), alpha.cpu().numpy(), rep, "bf16")
    sp2 = pamm.alloc_workspace(pamm.WS_COMPRESS, b, n, m, k, pamm.BF16)
    idx2, C2, invn2, f2, alpha2 = pamm.compress_fused(Xd, k, seed, sort_products=sp2)
    assert torch.equal(f, f2) and torch.equal(alpha, alpha2) and torch.equal(idx, idx2)
    need = pamm.workspace_bytes(pamm.WS_COMPRESS, b, n, m, k, pamm.BF16)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    rpb = max(64, (-(-b // sms) + 63) // 64 * 64)
    used = -(-b // rpb) * k * 4
    assert used <= need and torch.equal(sp[:used], sp2[:used])
    # ---- Z ----
    Zg = parity.to_f64(Z)
    assert Zg.shape == (b, m)
    if rows is None:
        Zo = orc.linear_forward(X, W)
        err = parity.rel_fro(Zg, Zo)
        parity.check_elementwise("Z", Zg, Zo, z_bound(X, W, Zo), rep)
    else:
        Zo = orc.linear_forward(X, W, rows=rows)
        err = parity.rel_fro(Zg[rows], Zo)
        parity.check_elementwise("Z", Zg[rows], Zo, z_bound(X, W, Zo, rows=rows), rep)
    assert err <= 2.0 ** -8, err                    # bf16 rounding of the output dominates: about 2^-9 / sqrt(3)
    rep.err["Z"] = err
    return rep, Z


# (b, n, m, k): ragged in every dimension; one and several column tiles; generators in one and in several chunks
SMALL = [
    (300, 72, 40, 16),
    (1000, 136, 264, 17),
    (777, 520, 1032, 128),
    (2500, 200, 776, 300),
    (129, 64, 8, 129),          # fewer than 256 rows: one CTA per tile
    (200, 200, 776, 48),        # the same, several column tiles
    (4133, 264, 520, 64),
    (256, 64, 264, 129),        # exactly one pair of row blocks; generators padded to two halves of 80
    (257, 136, 8, 33),          # the second pair holds one row
    (640, 72, 520, 513),        # three chunks of generators on pairs of CTAs
]


@pytest.mark.parametrize("b,n,m,k", SMALL)
def test_fused_forward_small_cases(b, n, m, k):
    X, _ = synth.random_case(b, n, 8, "bf16", seed=b + k, centres=max(2, k // 2))
    W = make_weight(n, m, seed=b)
    check_forward(X, W, k, seed=11 + k)


def test_fused_forward_with_padded_rows():
    X, _ = synth.random_case(700, 67, 8, "bf16", seed=4, centres=6)
    W = make_weight(67, 88, seed=2)
    check_forward(X, W, 24, seed=3, ldx=72)


def test_product_alone_without_generators():
    # k = 0: the layer's output only, e.g. when no gradient is wanted
    X, _ = synth.random_case(1111, 200, 8, "bf16", seed=21)
    W = make_weight(200, 392, seed=22)
    Xd, Wd = parity.to_device(X), parity.to_device(W)
    Z, *_ = pamm.linear_forward(Xd, Wd, 0)
    Zo = orc.linear_forward(X, W)
    rep = parity.Report(b=1111, k=0)
    parity.check_elementwise("Z", parity.to_f64(Z), Zo, z_bound(X, W, Zo), rep)
    # and the same bits as the fused call's Z
    Z2, *_ = pamm.linear_forward(Xd, Wd, 32, 5)
    assert torch.equal(Z, Z2)
    assert pamm.last_device_status() == pamm.OK


def test_fused_forward_is_bit_reproducible_and_rejects_what_it_does_not_serve():
    X, _ = synth.random_case(3000, 256, 8, "bf16", seed=31, centres=20)
    W = make_weight(256, 520, seed=32)
    Xd, Wd = parity.to_device(X), parity.to_device(W)
    outs = [pamm.linear_forward(Xd, Wd, 48, 5) for _ in range(3)]
    for o in outs[1:]:
        for a, b_ in zip(outs[0], o):
            assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a,
                               b_.view(torch.int16) if b_.dtype == torch.bfloat16 else b_)
    with pytest.raises(pamm.PammError) as e:
        pamm.linear_forward(Xd.float(), Wd.float(), 48, 5)                 # fp32: no tensor-core kernel, no stand-in
    assert e.value.code == pamm.ERR_UNSUPPORTED
    with pytest.raises(pamm.PammError):
        pamm.linear_forward(Xd, Wd, 5, 5)                                  # fewer than 16 generators


@pytest.mark.parametrize("name", ["c2", "c4"])
def test_fused_forward_full_size(name):
    # Z at full size on sampled rows the oracle computes one by one; f and alpha through the usual full checks
    inp = synth.make_inputs(name, with_dY=False)
    w = inp.workload
    W = make_weight(w.n, w.m, seed=w.seed)
    rows = np.sort(np.random.default_rng(7).choice(inp.b, size=96, replace=False))
    rows[0], rows[-1] = 0, inp.b - 1
    rep, Z = check_forward(inp.X, W, w.ks[0], seed=w.index_seed, rows=rows)
    parity.record(f"{name} fused forward k={w.ks[0]}", rep)
    # every row block and column tile was written: no element of Z is left at its initial value
    assert torch.isfinite(Z.float()).all()


@pytest.mark.parametrize("b,n,m", [(1111, 200, 392), (300, 72, 40), (129, 64, 264), (4133, 520, 264), (256, 1032, 776)])
def test_input_gradient_product(b, n, m):
    # dX = dZ W^T (Algorithm 3) through the forward kernel with W as the operand whose contraction index is contiguous;
    # the oracle's plain product of dZ with the transposed weight is the definition
    dZ, _ = synth.random_case(b, m, 8, "bf16", seed=b + m)
    W = make_weight(n, m, seed=n)
    dX = pamm.linear_backward_input(parity.to_device(dZ), parity.to_device(W))
    Wt = np.ascontiguousarray(W.T)
    ref = orc.linear_forward(dZ, Wt)
    rep = parity.Report(b=b, k=0)
    parity.check_elementwise("dX", parity.to_f64(dX), ref, z_bound(dZ, Wt, ref), rep)
    assert pamm.last_device_status() == pamm.OK
    with pytest.raises(pamm.PammError) as e:
        pamm.linear_backward_input(parity.to_device(dZ).float(), parity.to_device(W).float())
    assert e.value.code == pamm.ERR_UNSUPPORTED
