"""pvt_vstep_block: the V step over the layers of a block in one call against the CPU checker layer by layer."""
import numpy as np
import pytest
import torch

import helpers
from oracle import pvt_oracle as oracle
from paper_2405_14852_b200 import binding as B
from paper_2405_14852_b200 import synth
from paper_2405_14852_b200.vstep import VStepLayer

pytestmark = pytest.mark.gpu


def oracle_nearest(X, C):
    return oracle.encode(X, C[None], np.zeros((X.shape[0], 1))).codes[:, 0]


def test_block_of_mixed_layers_against_the_checker():
    """Four layers of different shapes and representations (one large fp16 codebook on the tensor engine, a small
    fp32 codebook, two additive codebooks, three additive codebooks) share one workspace and one call."""
    specs = [dict(rows=256, cols=512, M=1, K=4096, f16=True, tau="0.05"),
             dict(rows=100, cols=264, M=1, K=64, f16=False, tau="0.2"),
             dict(rows=96, cols=136, M=2, K=256, f16=True, tau="0.1"),
             dict(rows=64, cols=128, M=3, K=32, f16=True, tau="1.0")]
    hosts, devs, ks, idxs, outs = [], [], [], [], []
    for i, sp in enumerate(specs):
        L = synth.make_layer(sp["rows"], sp["cols"], cfg=300 + i, num_codebooks=sp["M"], codebook_size=sp["K"],
                             codebook_fp16=sp["f16"], nearest=oracle_nearest)
        hosts.append(L)
        dev = VStepLayer.from_host(L)
        devs.append(dev)
        k = synth.subspace_size(sp["tau"], L.num_groups)
        ks.append(k)
        idxs.append(torch.full((k,), -1, dtype=torch.int32, device="cuda"))
        outs.append(torch.empty(L.rows, L.cols, dtype=torch.float16, device="cuda"))
    block = B.Block([d.desc for d in devs], ks, idxs, outs)
    ws = torch.empty(block.workspace_bytes(), dtype=torch.uint8, device="cuda")
    B.pvt_workspace_init(ws)
    B.pvt_vstep_block(block, ws)
    torch.cuda.synchronize()
    assert B.pvt_status(ws) == 0
    for L, dev, k, idx, out in zip(hosts, devs, ks, idxs, outs):
        M, G = L.num_codebooks, L.num_groups
        want = oracle.vstep(L.W, L.g, L.scale, L.codebooks, L.codes, L.eta, k, L.beam)
        assert np.array_equal(idx.cpu().numpy().astype(np.uint32), want.idx)
        got = dev.codes.cpu().numpy().reshape(G, M)
        sel = want.idx.astype(np.int64)
        helpers.check_codes_against_oracle(want.t, L.codebooks, got[sel], want.enc, 1e-6)
        rest = np.ones(G, bool)
        rest[sel] = False
        assert np.array_equal(got[rest], L.codes.reshape(G, M)[rest])
        want_W = oracle.dequant(got, L.codebooks, L.scale, L.rows, L.cols).astype(np.float16)
        assert out.cpu().numpy().tobytes() == want_W.tobytes()


def test_block_without_dequantisation_and_with_skipped_outputs():
    L = synth.make_layer(64, 256, cfg=310, codebook_size=128, codebook_fp16=True)
    devs = [VStepLayer.from_host(L), VStepLayer.from_host(L)]
    k = 50
    idxs = [torch.empty(k, dtype=torch.int32, device="cuda") for _ in devs]
    out = torch.zeros(64, 256, device="cuda")
    for W_hats in (None, [None, out]):
        block = B.Block([d.desc for d in devs], [k, k], idxs, W_hats)
        ws = torch.empty(block.workspace_bytes(), dtype=torch.uint8, device="cuda")
        B.pvt_workspace_init(ws)
        B.pvt_vstep_block(block, ws)
        torch.cuda.synchronize()
        assert B.pvt_status(ws) == 0
    assert torch.equal(idxs[0], idxs[1])
    want = oracle.dequant(devs[1].codes.cpu().numpy(), L.codebooks, L.scale, 64, 256)
    assert out.cpu().numpy().tobytes() == want.tobytes()
