"""The seeded generators: determinism, subset consistency, and the stated distributions."""
import numpy as np
import torch

from paper_2609_12399_b200 import inputs


def test_workloads_match_benchmark_configs():
    w = inputs.WORKLOADS
    assert [(x.R, x.L, x.H, x.dk, x.W, x.D) for x in w] == [
        (1, 1, 2, 32, 8, 3), (1, 1, 16, 128, 128, 4), (1, 1, 32, 128, 512, 4),
        (8, 1, 32, 128, 1024, 6), (4, 16, 32, 128, 512, 8)]
    assert w[0].record_bytes == 264 and all(x.record_bytes == 520 for x in w[1:])
    assert [x.prompt_len for x in w] == [64, 4096, 16384, 8192, 16384]


def test_deterministic_and_subsets_consistent():
    wl = inputs.WORKLOADS[1]
    a = inputs.decode_token(wl, 0, 0, 2)
    b = inputs.decode_token(wl, 0, 0, 2)
    for n in a:
        assert torch.equal(a[n], b[n])
    beams, heads = [5, 100, 17], [3, 15]
    s = inputs.decode_token(wl, 0, 0, 2, beams=beams, heads=heads)
    for n in a:
        assert torch.equal(s[n], a[n][beams][:, heads])
    q = inputs.decode_query(wl, 0, 0, 2)
    assert torch.equal(inputs.decode_query(wl, 0, 0, 2, beams=beams, heads=heads), q[beams][:, heads])
    p = inputs.prompt_tokens(wl, 0, 0, 10, 20, heads=heads)
    full = inputs.prompt_tokens(wl, 0, 0, 0, 32)
    for n in p:
        assert torch.equal(p[n], full[n][10:20][:, heads])
    # different step / request / layer / kind give different draws
    assert not torch.equal(a["k"], inputs.decode_token(wl, 0, 0, 1)["k"])
    assert not torch.equal(a["k"], a["v"][..., : wl.dk])
    assert not torch.equal(a["k"], q)


def test_distributions():
    wl = inputs.WORKLOADS[2]
    t = inputs.decode_token(wl, 0, 0, 1)
    assert t["k"].dtype == torch.bfloat16 and t["alpha"].dtype == torch.float32
    kn = t["k"].double().norm(dim=-1)
    assert (kn - 1).abs().max() < 2e-2                  # unit before bf16 rounding
    v = t["v"].double()
    assert abs(v.mean()) < 5e-3 and abs(v.std() - 1) < 5e-3
    assert t["alpha"].min() >= 0.9 and t["alpha"].max() <= 1.0 and abs(t["alpha"].mean() - 0.95) < 2e-3
    assert 0 < t["beta"].min() and t["beta"].max() < 1 and abs(t["beta"].mean() - 0.5) < 5e-3
    z = torch.log(t["beta"].double() / (1 - t["beta"].double()))       # logit(beta) ~ N(0,1)
    assert abs(z.std() - 1) < 2e-2
    t0 = inputs.decode_token(inputs.WORKLOADS[0], 0, 0, 0)
    assert t0["k"].dtype == torch.float32 and (t0["k"].double().norm(dim=-1) - 1).abs().max() < 1e-6


def test_parents_uniform_and_zipf():
    u = inputs.parents(inputs.WORKLOADS[3], 0, 1)
    assert u.dtype == torch.int32 and u.shape == (1024,) and 0 <= u.min() and u.max() < 1024
    assert 600 < len(torch.unique(u)) < 700             # ~ W (1 - 1/e) = 647 distinct parents
    z = inputs.parents(inputs.WORKLOADS[2], 0, 1)
    assert 0 <= z.min() and z.max() < 512
    nz = len(torch.unique(z))
    assert 90 < nz < 180                                # Zipf(1.2): far fewer distinct parents
    z4 = inputs.parents(inputs.WORKLOADS[4], 0, 1)
    assert len(torch.unique(z4)) < nz
    counts = torch.bincount(z.long(), minlength=512).double().sort(descending=True).values
    assert counts[0] / 512 > 0.12                       # the top-ranked parent takes ~ 1/H_{512,1.2} = 0.22 -> loose
    assert not torch.equal(z, inputs.parents(inputs.WORKLOADS[2], 0, 2))
    assert inputs.parents(inputs.WORKLOADS[2], 0, 1, W_prev=7, W_new=3).max() < 7
