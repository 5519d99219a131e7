"""Config 2 at its full size (1,000,000 flows) in the launch configuration the benchmark
times: features, fast-model probabilities, routing and the assigned-id list are compared
with the oracle on ALL flows (bit-exact); wide rows and slow-model logits on sampled rows
that include the first and the last GEMM row tile."""
import numpy as np
import pytest

import flowgen
import oracle
from workload import make_workload

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def bits(a):
    return np.ascontiguousarray(a, np.float32).view(np.uint32)


def test_config2_full_size_against_oracle():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2402_03694_b200 import build, binding as sf, harness as hz
    build.build()
    cfg = flowgen.get_config(2)
    n = cfg.n
    wl = make_workload(cfg, n=n, threads=16)
    feat = oracle.extract_features(wl["fast"], cfg.N, cfg.F, threads=16)
    prob = oracle.forest_infer(wl["forest"], feat, threads=16)
    rt = oracle.route_lc(prob, wl["tau"])
    k = rt["n_esc"]
    assert 0.2 < k / n < 0.28

    ctx = sf.sf_ctx_create(0, 0)
    forest = hz.make_forest(ctx, wl["forest"])
    slow = hz.make_slow(ctx, cfg, wl["slow"])
    fast_d = hz.upload_packets(wl["fast"], with_hdr=False)
    wide_d = hz.upload_packets(wl["wide"])
    rcfg = hz.route_cfg_for(cfg, hz.dev(wl["tau"]), n)
    label = torch.zeros(n, dtype=torch.uint8, device="cuda")
    stage = torch.zeros(n, dtype=torch.uint8, device="cuda")
    n_esc = torch.zeros(1, dtype=torch.uint32, device="cuda")
    sf.sf_serve_batch(ctx, forest, slow, fast_d["struct"], cfg.N, cfg.F, wide_d["struct"], rcfg, label, stage, n_esc)
    torch.cuda.synchronize()
    c = sf.sf_ctx_poll(ctx, reset=True)
    assert c.device_error == 0 and int(n_esc.cpu().numpy()[0]) == k and c.n_slow_done == k
    p = sf.sf_serve_batch_intermediates(ctx)
    assert np.array_equal(bits(hz.ptr_tensor(p["feat"], (n, cfg.F), torch.float32).cpu().numpy()), bits(feat))
    assert np.array_equal(bits(hz.ptr_tensor(p["fast_out"], (n, cfg.C), torch.float32).cpu().numpy()), bits(prob))
    assert np.array_equal(hz.ptr_tensor(p["esc_ids"], (k,), torch.uint32).cpu().numpy(), rt["esc_ids"])
    st = stage.cpu().numpy()
    assert np.array_equal(st, 1 + rt["decision"])
    lab = label.cpu().numpy()
    assert np.array_equal(lab[st == 1], rt["label"][st == 1])
    # sampled rows: first tile, last (ragged) tile, and a random spread
    rng = np.random.default_rng(0)
    sel = np.unique(np.concatenate([np.arange(128), np.arange(k - 128, k), rng.integers(0, k, 256)]))
    rows_ref = oracle.wide_rows(0, rt["esc_ids"][sel], wl["wide"], cfg.P, True, threads=16)
    rows_gpu = hz.ptr_tensor(p["rows"], (k, cfg.D), torch.bfloat16)[torch.from_numpy(sel).cuda()].float().cpu().numpy()
    assert np.array_equal(bits(rows_gpu), bits(rows_ref))
    logits_ref, label_ref = oracle.mlp(wl["slow"], rows_ref, True, threads=16)
    logits_gpu = hz.ptr_tensor(p["logits"], (k, cfg.n_slow_classes), torch.float32).cpu().numpy()[sel]
    assert np.max(np.abs(logits_gpu - logits_ref)) <= 2e-2
    s = np.sort(logits_ref, axis=1)
    clear = (s[:, -1] - s[:, -2]) >= 4e-2
    assert np.array_equal(lab[rt["esc_ids"][sel]][clear], label_ref[clear])
    sf.sf_slow_destroy(slow); sf.sf_forest_destroy(forest); sf.sf_ctx_destroy(ctx)
