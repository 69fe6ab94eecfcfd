"""Token-subset gather / scatter against the oracle (exact), and attention over a pruned token subset."""
import numpy as np
import pytest
import torch

import oracle
import _util as U
from paper_2606_23743_b200 import binding as B
from paper_2606_23743_b200.workloads import WORKLOADS, shrink

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.uint8, torch.float32])
def test_gather_and_scatter_are_exact(dtype):
    g = torch.Generator().manual_seed(11)
    Bq, H, N, d = 2, 3, 777, 128
    x = torch.randint(0, 255, (Bq, H, N, d), generator=g, dtype=torch.uint8)
    if dtype != torch.uint8:
        x = x.to(dtype)
    idx = torch.stack([torch.randperm(N, generator=g)[:400].sort().values for _ in range(Bq)]).to(torch.int32)
    xd, idxd = x.cuda(), idx.cuda()
    out = torch.full((Bq, H, 400, d), 9, dtype=dtype, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.gather_tokens(xd, idxd, out, st)
    torch.cuda.synchronize()
    xn = x.view(torch.uint16).numpy() if dtype == torch.bfloat16 else x.numpy()
    ref = oracle.gather_tokens(xn, idx.numpy())
    got = out.cpu()
    got = got.view(torch.uint16).numpy() if dtype == torch.bfloat16 else got.numpy()
    np.testing.assert_array_equal(got, ref)
    assert int(st.item()) == 0
    # scatter back into a buffer of sevens
    full = torch.full((Bq, H, N, d), 7, dtype=dtype, device="cuda")
    B.scatter_tokens(out, idxd, full, st)
    torch.cuda.synchronize()
    fulln = np.full(xn.shape, 0, xn.dtype)
    sevens = torch.full((1,), 7, dtype=dtype)
    fulln[...] = sevens.view(torch.uint16).numpy()[0] if dtype == torch.bfloat16 else sevens.numpy()[0]
    ref2 = oracle.scatter_tokens(ref, idx.numpy(), fulln)
    got2 = full.cpu()
    got2 = got2.view(torch.uint16).numpy() if dtype == torch.bfloat16 else got2.numpy()
    np.testing.assert_array_equal(got2, ref2)


def test_strided_source_and_bad_index():
    g = torch.Generator().manual_seed(12)
    qkv = torch.randn(1, 2, 300, 3 * 128, generator=g).to(torch.bfloat16).cuda()     # packed QKV rows
    k = qkv[..., 128:256]
    idx = torch.tensor([[5, 299, 0, 17, 1000]], dtype=torch.int32).cuda()             # last index is out of range
    out = torch.zeros(1, 2, 5, 128, dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.gather_tokens(k, idx, out, st)
    torch.cuda.synchronize()
    assert int(st.item()) & B.SVA_DEV_BAD_INDEX
    assert torch.equal(out[:, :, :4], k[:, :, [5, 299, 0, 17]]) and (out[:, :, 4] == 0).all()


def test_attention_over_a_pruned_token_subset():
    """Half of the tokens kept (per batch item), gathered, routed and attended as a sequence of its own,
    output scattered back: equals the oracle run on the oracle-gathered inputs; pruned rows untouched."""
    w_full = shrink(WORKLOADS["medium"], H=2, T=4)                 # N = 4096
    (q, k, v), (qb, kb, vb) = U.host_inputs(w_full)
    g = torch.Generator().manual_seed(13)
    M = w_full.N // 2 - 24                                         # ragged: 2024 kept tokens
    idx = torch.stack([torch.randperm(w_full.N, generator=g)[:M].sort().values for _ in range(w_full.B)]).to(torch.int32)
    idxd = idx.cuda()
    qd, kd, vd = U.dev(q), U.dev(k), U.dev(v)
    n_alloc = -(-M // 128) * 128
    sub = [torch.zeros(w_full.B, w_full.H, n_alloc, w_full.d, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    for src, dst in zip((qd, kd, vd), sub):
        B.gather_tokens(src, idxd, dst)
    w = shrink(w_full, T=1, Hg=1, Wg=M, k=6)                       # the gathered sequence: N = M, Nb = 16
    assert w.N == M
    rp, ci, _ = U.gpu_select(w, sub[0], sub[1])
    o, lse, st = U.gpu_attn(w, sub[0], sub[1], sub[2], rp, ci)
    assert st == 0
    qs, ks_, vs = (oracle.gather_tokens(x[:, :, :w_full.N], idx.numpy()) for x in (qb, kb, vb))
    pad = lambda a: np.concatenate([a, np.zeros((a.shape[0], a.shape[1], n_alloc - M, a.shape[3]), a.dtype)], axis=2)
    sel, _ = U.oracle_select(w, pad(qs), pad(ks_))
    n_diff, n_near = U.compare_selection(sel, rp, ci)
    assert n_diff <= n_near
    U.check_attn_vs_oracle(w, pad(qs), pad(ks_), pad(vs), rp, ci, o, lse, list(range(w.R)))
    full = torch.full((w_full.B, w_full.H, w_full.N, w_full.d), 7.0, dtype=torch.bfloat16, device="cuda")
    B.scatter_tokens(o[:, :, :M].contiguous(), idxd, full)
    torch.cuda.synchronize()
    kept = torch.zeros(w_full.N, dtype=torch.bool); kept[idx[0].long()] = True
    assert torch.equal(full[0][:, kept.cuda()], o[0, :, :M]) and (full[0][:, (~kept).cuda()] == 7.0).all()
