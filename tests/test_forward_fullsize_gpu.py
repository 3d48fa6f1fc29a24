"""Parity at the full benchmark sizes, in the launch configuration bench.py times: the whole
workload runs on the GPU through mxattn_forward_ws and sampled output rows (rows are independent
in Algorithm 2) are compared with the oracle, which computes them one by one."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import attention
from tests import util

pytestmark = pytest.mark.gpu


def sampled_rows(cfg, head, n_random=10):
    rng = np.random.default_rng([4242, head])
    fixed = [0, 127, 128, cfg.Nq - 1, cfg.Nq - 2, (cfg.Nq - 1) // 128 * 128, (cfg.Nq - 1) // 256 * 256, cfg.Nq // 2]
    rows = set(r for r in fixed if 0 <= r < cfg.Nq) | set(rng.integers(0, cfg.Nq, n_random).tolist())
    return np.array(sorted(rows))


@pytest.mark.parametrize("name,heads", [("outlier", [0, 7, 15, 23]), ("wan22", [0, 13, 26, 39]), ("hunyuan", [0, 8, 16, 23]),
                                        ("wan22_cross", [0, 13, 26, 39])])
@pytest.mark.parametrize("variant", ["uos_pnq", "ocp_direct"])
def test_full_size_config_sampled_rows(name, heads, variant):
    import paper_2607_24377_b200 as mx
    if variant == "ocp_direct" and name not in ("outlier", "wan22_cross"):
        pytest.skip("the vanilla variant is checked at full size on the small-KV configs only (time)")
    cfg = si.CONFIGS[name]
    uos = pnq = (variant == "uos_pnq")
    B, H, Nq, Nkv, d = cfg.B, cfg.H, cfg.Nq, cfg.Nkv, cfg.d
    hq = np.empty((B, H, Nq, d), np.uint16); hk = np.empty((B, H, Nkv, d), np.uint16); hv = np.empty((B, H, Nkv, d), np.uint16)
    for h in range(H):
        hq[0, h], hk[0, h], hv[0, h] = si.make_head(cfg, 0, h)
    dq, dk, dv = util.to_dev_bf16(hq), util.to_dev_bf16(hk), util.to_dev_bf16(hv)
    out = torch.empty((B, H, Nq, d), dtype=torch.float32, device="cuda")
    ws = torch.empty(mx.forward_workspace_bytes(B, H, Nq, Nkv, d), dtype=torch.uint8, device="cuda")
    flags = (mx.FLAG_UOS if uos else 0) | (mx.FLAG_PNQ if pnq else 0) | mx.FLAG_OUT_FP32
    mx.forward_ws(dq, dk, dv, out, B, H, Nq, Nkv, d, cfg.softmax_scale, flags, ws)
    assert mx.device_status(ws) == 0
    f = util.bits_to_f64
    num = den = 0.0
    worst = 0.0
    for h in heads:
        rows = sampled_rows(cfg, h)
        want = attention.forward_head(f(hq[0, h]), f(hk[0, h]), f(hv[0, h]), cfg.softmax_scale, uos, pnq, rows=rows)
        got = out[0, h][torch.from_numpy(rows).cuda()].double().cpu().numpy()
        assert np.isfinite(got).all()
        num += float(((got - want) ** 2).sum()); den += float((want ** 2).sum())
        worst = max(worst, float(np.abs(got - want).max()))
    rel = (num / den) ** 0.5
    assert rel <= 1e-3 and worst <= 4e-3, (name, variant, rel, worst)
    # whole-output property that holds at any size: every output element is finite and bounded by max |V-hat| <= 6 * 2^e
    assert bool(torch.isfinite(out).all())
