"""The layer pieces around the projections (RMSNorm, rotary embedding, SiLU gate, add) against the
layer oracle's definitions in fp64; the backward entry points against autograd of those definitions."""
import numpy as np
import pytest
import torch

from oracle import layer_oracle as lo
from paper_2607_28848_b200 import layer_ops as mo

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def bf(t):
    return t.to(torch.bfloat16)


def close(got, ref, tol=1.2e-2):
    got, ref = got.double().cpu(), ref.double()
    assert float(((got - ref).abs() - tol * (1 + ref.abs())).max()) <= 0, float((got - ref).abs().max())


@pytest.mark.parametrize("rows,d", [(1, 8), (37, 512), (130, 4096), (5, 14336)])
def test_rmsnorm_forward_and_backward(rows, d):
    g = torch.Generator().manual_seed(rows + d)
    x = bf(torch.randn(rows, d, generator=g) * 1.7).to(DEV)
    gain = (1 + 0.2 * torch.randn(d, generator=g)).float().to(DEV)
    dy = bf(torch.randn(rows, d, generator=g)).to(DEV)
    y, dx = torch.empty_like(x), torch.empty_like(x)
    mo.mlora_rmsnorm_forward(x, gain, y)
    mo.mlora_rmsnorm_backward(x, gain, dy, dx)
    xr = x.double().cpu().requires_grad_(True)
    yr = lo.rmsnorm(xr, gain.double().cpu())
    yr.backward(dy.double().cpu())
    close(y, yr.detach())
    close(dx, xr.grad)


@pytest.mark.parametrize("heads,dh", [(4, 128), (32, 128), (8, 64), (1, 16)])
def test_rope_forward_and_transpose(heads, dh):
    g = torch.Generator().manual_seed(heads * dh)
    T = 77
    x = bf(torch.randn(T, heads * dh, generator=g)).to(DEV)
    pos = torch.randint(0, 4000, (T,), generator=g, dtype=torch.int32).to(DEV)
    y = torch.empty_like(x)
    mo.mlora_rope(x, y, pos, heads, dh)
    ref = lo.rope(x.double().cpu().reshape(T, heads, dh), pos.cpu().long()).reshape(T, heads * dh)
    close(y, ref)
    # the transposed rotation undoes the forward (up to the two bf16 roundings) and is its input gradient
    back = torch.empty_like(x)
    mo.mlora_rope(y, back, pos, heads, dh, transpose=True)
    close(back, x.double().cpu(), tol=2e-2)
    xr = x.double().cpu().reshape(T, heads, dh).requires_grad_(True)
    dy = bf(torch.randn(T, heads * dh, generator=g))
    lo.rope(xr, pos.cpu().long()).backward(dy.double().reshape(T, heads, dh))
    dx = torch.empty_like(x)
    mo.mlora_rope(dy.to(DEV), dx, pos, heads, dh, transpose=True)
    close(dx, xr.grad.reshape(T, heads * dh))
    mo.mlora_rope(x, x, pos, heads, dh)                      # in place
    assert torch.equal(x, y)


@pytest.mark.parametrize("n", [8, 4096 * 33, 14336 * 70])
def test_swiglu_and_add(n):
    g = torch.Generator().manual_seed(n)
    a, b, d = (bf(torch.randn(n, generator=g) * 2).to(DEV) for _ in range(3))
    m, dg, du, s = (torch.empty_like(a) for _ in range(4))
    mo.mlora_swiglu_forward(a, b, m)
    mo.mlora_swiglu_backward(a, b, d, dg, du)
    mo.mlora_add(a, b, s)
    ar, br = a.double().cpu().requires_grad_(True), b.double().cpu().requires_grad_(True)
    mr = torch.nn.functional.silu(ar) * br
    mr.backward(d.double().cpu())
    close(m, mr.detach())
    close(dg, ar.grad)
    close(du, br.grad)
    close(s, a.double().cpu() + b.double().cpu())


@pytest.mark.parametrize("heads,kv,dh", [(4, 2, 128), (8, 8, 64), (6, 1, 128)])
def test_attention_forward_and_backward(heads, kv, dh):
    g = torch.Generator().manual_seed(heads * 100 + kv)
    lens = [1, 37, 5, 130, 1, 64]                                  # packed sequences, decode-like single rows among them
    T = sum(lens)
    q = bf(torch.randn(T, heads * dh, generator=g)).to(DEV)
    k = bf(torch.randn(T, kv * dh, generator=g)).to(DEV)
    v = bf(torch.randn(T, kv * dh, generator=g)).to(DEV)
    dO = bf(torch.randn(T, heads * dh, generator=g)).to(DEV)
    start, end, seqs, r = [], [], [], 0
    for n in lens:
        start += [r] * n; end += [r + n] * n; seqs.append(list(range(r, r + n))); r += n
    ss, se = torch.tensor(start, dtype=torch.int32, device=DEV), torch.tensor(end, dtype=torch.int32, device=DEV)
    o, dq = torch.empty_like(q), torch.empty_like(q)
    dk, dv = torch.empty_like(k), torch.empty_like(v)
    lse = torch.empty((T, heads), dtype=torch.float32, device=DEV)
    mo.mlora_attention_forward(q, k, v, o, lse, ss, se, heads, kv, dh)
    mo.mlora_attention_backward(q, k, v, o, lse, dO, dq, dk, dv, ss, se, heads, kv, dh)
    qr = q.double().cpu().reshape(T, heads, dh).requires_grad_(True)
    kr = k.double().cpu().reshape(T, kv, dh).requires_grad_(True)
    vr = v.double().cpu().reshape(T, kv, dh).requires_grad_(True)
    orf = lo.attention(qr, kr, vr, seqs)
    orf.backward(dO.double().cpu().reshape(T, heads, dh))
    close(o, orf.detach().reshape(T, heads * dh))
    close(dq, qr.grad.reshape(T, heads * dh), tol=2e-2)
    close(dk, kr.grad.reshape(T, kv * dh), tol=2e-2)
    close(dv, vr.grad.reshape(T, kv * dh), tol=2e-2)


@pytest.mark.parametrize("lens", [[1], [127], [128], [129], [300, 5, 1, 1, 200], [64] * 9, [1] * 140, [700]])
@pytest.mark.parametrize("heads,kv", [(4, 2), (3, 1)])
def test_attention_tensor_core_kernels(lens, heads, kv):
    """Head size 128 (the tcgen05 kernel): query tiles that hold one sequence, several sequences or a
    ragged last tile; sequences longer than one key block (online softmax over several blocks);
    outputs and log-sum-exp against the fp64 definition."""
    dh = 128
    g = torch.Generator().manual_seed(sum(lens) * 10 + heads)
    T = sum(lens)
    q = bf(torch.randn(T, heads * dh, generator=g) * 2.0).to(DEV)     # a wider score range than unit inputs give
    k = bf(torch.randn(T, kv * dh, generator=g)).to(DEV)
    v = bf(torch.randn(T, kv * dh, generator=g)).to(DEV)
    start, end, seqs, r = [], [], [], 0
    for n in lens:
        start += [r] * n; end += [r + n] * n; seqs.append(list(range(r, r + n))); r += n
    ss, se = torch.tensor(start, dtype=torch.int32, device=DEV), torch.tensor(end, dtype=torch.int32, device=DEV)
    o = torch.full_like(q, float("nan"))
    lse = torch.full((T, heads), float("nan"), dtype=torch.float32, device=DEV)
    mo.mlora_attention_forward(q, k, v, o, lse, ss, se, heads, kv, dh)
    assert mo.mlora_layer_ops_poll_status() == 0
    qr, kr, vr = (x.double().cpu() for x in (q, k, v))
    ref = lo.attention(qr.reshape(T, heads, dh), kr.reshape(T, kv, dh), vr.reshape(T, kv, dh), seqs)
    close(o, ref.reshape(T, heads * dh))
    # log-sum-exp of the scaled scores of every row, from the definition
    rep = heads // kv
    lse_ref = torch.empty(T, heads, dtype=torch.float64)
    for rows in seqs:
        for h in range(heads):
            sc = qr.reshape(T, heads, dh)[rows, h] @ kr.reshape(T, kv, dh)[rows, h // rep].T / dh ** 0.5
            sc = sc.masked_fill(torch.triu(torch.ones(len(rows), len(rows), dtype=torch.bool), 1), float("-inf"))
            lse_ref[rows, h] = torch.logsumexp(sc, dim=1)
    assert torch.allclose(lse.double().cpu(), lse_ref, rtol=0, atol=2e-3), float((lse.double().cpu() - lse_ref).abs().max())
    # the gradients (tcgen05 kernels as well): dq per query tile, dk and dv per key tile over the heads of the group
    dO = bf(torch.randn(T, heads * dh, generator=g)).to(DEV)
    dq = torch.full_like(q, float("nan"))
    dk, dv = torch.full_like(k, float("nan")), torch.full_like(v, float("nan"))
    mo.mlora_attention_backward(q, k, v, o, lse, dO, dq, dk, dv, ss, se, heads, kv, dh)
    assert mo.mlora_layer_ops_poll_status() == 0
    qg = qr.reshape(T, heads, dh).clone().requires_grad_(True)
    kg = kr.reshape(T, kv, dh).clone().requires_grad_(True)
    vg = vr.reshape(T, kv, dh).clone().requires_grad_(True)
    lo.attention(qg, kg, vg, seqs).backward(dO.double().cpu().reshape(T, heads, dh))
    # P and dS enter the tensor cores rounded to bf16 (relative 2^-9 per term, up to 128 terms per block):
    # with the doubled queries of this test dS reaches ~10, so the bound is 3e-2 here (2e-2 at unit scale above)
    close(dq, qg.grad.reshape(T, heads * dh), tol=3e-2)
    close(dk, kg.grad.reshape(T, kv * dh), tol=3e-2)
    close(dv, vg.grad.reshape(T, kv * dh), tol=3e-2)


@pytest.mark.parametrize("seed", range(6))
def test_attention_random_sequence_mixes(seed):
    """Seeded random packed batches (one to eleven sequences of 1 to 600 rows, several head groupings),
    forward and gradients of the head-size-128 kernels against the fp64 definition and its autograd."""
    import numpy as np
    rng = np.random.default_rng(900 + seed)
    n_seq = int(rng.integers(1, 12))
    lens = [int(x) for x in (rng.integers(1, 40, n_seq) if seed % 3 == 0 else rng.integers(1, 600, n_seq))]
    heads, kv = [(4, 2), (8, 1), (2, 2), (6, 3)][int(rng.integers(0, 4))]
    dh, T = 128, sum(lens)
    g = torch.Generator().manual_seed(seed)
    q, k, v, dO = (bf(torch.randn(T, n * dh, generator=g)).to(DEV) for n in (heads, kv, kv, heads))
    start, end, seqs, r = [], [], [], 0
    for n in lens:
        start += [r] * n; end += [r + n] * n; seqs.append(list(range(r, r + n))); r += n
    ss, se = torch.tensor(start, dtype=torch.int32, device=DEV), torch.tensor(end, dtype=torch.int32, device=DEV)
    o, dq = torch.full_like(q, float("nan")), torch.full_like(q, float("nan"))
    dk, dv = torch.full_like(k, float("nan")), torch.full_like(v, float("nan"))
    lse = torch.empty((T, heads), dtype=torch.float32, device=DEV)
    mo.mlora_attention_forward(q, k, v, o, lse, ss, se, heads, kv, dh)
    mo.mlora_attention_backward(q, k, v, o, lse, dO, dq, dk, dv, ss, se, heads, kv, dh)
    assert mo.mlora_layer_ops_poll_status() == 0
    qr = q.double().cpu().reshape(T, heads, dh).requires_grad_(True)
    kr = k.double().cpu().reshape(T, kv, dh).requires_grad_(True)
    vr = v.double().cpu().reshape(T, kv, dh).requires_grad_(True)
    ref = lo.attention(qr, kr, vr, seqs)
    ref.backward(dO.double().cpu().reshape(T, heads, dh))
    close(o, ref.detach().reshape(T, heads * dh))
    close(dq, qr.grad.reshape(T, heads * dh), tol=2e-2)
    close(dk, kr.grad.reshape(T, kv * dh), tol=2e-2)
    close(dv, vr.grad.reshape(T, kv * dh), tol=2e-2)


def test_argument_errors():
    x = torch.zeros(4, 12, dtype=torch.bfloat16, device=DEV)           # 12 is not a multiple of 8
    gain = torch.ones(12, device=DEV)
    from paper_2607_28848_b200 import binding as mb
    with pytest.raises(mb.MloraError) as e:
        mo.mlora_rmsnorm_forward(x, gain, torch.empty_like(x))
    assert e.value.status == mb.MLORA_ERR_UNSUPPORTED
    with pytest.raises(mb.MloraError):
        mo.mlora_rope(x, x, torch.zeros(4, dtype=torch.int32, device=DEV), 1, 12)
