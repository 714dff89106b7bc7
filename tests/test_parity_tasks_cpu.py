"""CPU check of the test harness itself: the per-layer comparison task, the end-to-end task and the storage
control run on results that were made from the oracle (rounded the way the library stores them), directly and
through the spawn pool.  A correct "implementation" built that way must pass, and a planted mistake must fail."""
import numpy as np
import torch

import synth_inputs as si
from oracle import sepconv_oracle as O
from tests import parity_util as U


def t16(a, dtype):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(U.TD[dtype])


def fake_layer_task(L, dtype, x, lengths, p, g, index=0, spoil=None):
    S = O.block_fwd(L, x, lengths, p)
    G = O.block_bwd(L, g, lengths, p, S)
    dx = G["dx"] + G.get("dx_res", 0.0)
    saved = {"u": t16(S["u"], "f16"), "v": t16(S["v"], "f16"), "mean": torch.tensor(S["mean"], dtype=torch.float32),
             "invstd": torch.tensor(S["invstd"], dtype=torch.float32)}
    if L.residual == "proj":
        saved["vr"] = t16(S["vr"], "f16")
    y = S["y"] if spoil != "y" else S["y"] * 1.1
    return dict(index=index, L=L, dtype=dtype, x=t16(x, dtype), lengths=np.asarray(lengths), params=p, x_res=None,
                out_len=S["out_len"], saved=saved, pd={k: torch.tensor(v, dtype=torch.float32) for k, v in p.items()},
                y=t16(y, dtype), g=t16(g, dtype), dx=t16(dx, dtype), dx_res=None, dx_add=None, want_res=False,
                grads={"d" + k: torch.tensor(G["d" + k], dtype=torch.float32) for k in p})


def _draw(L, B, T, dtype, seed):
    d = si.draw(si.Workload("t", dtype, B, T, [L], seed, len_lo=T // 3, len_hi=T, affine="random"))
    return d.x, d.lengths, d.params[0], d.g


def test_layer_task_direct_and_in_pool():
    L = si.LayerCfg(12, 16, K=5, residual="proj")
    x, lengths, p, g = _draw(L, 3, 40, "bf16", 5)
    ok = fake_layer_task(L, "bf16", x, lengths, p, g, index=0)
    bad = fake_layer_task(L, "bf16", x, lengths, p, g, index=1, spoil="y")
    r = U.layer_task(ok)
    assert max(e for _, e in r["rows"]) <= 1.0 and r["hard"] == 0
    with U.make_pool(workers=2, blas_threads=1) as pool:
        out = pool.map(U.layer_task, [ok, bad], chunksize=1)
    assert out[0]["rows"] == r["rows"]
    assert dict(out[1]["rows"])["y"] > 1.0            # the planted 10 % error is caught


def test_end_to_end_and_control_tasks():
    w = si.tiny_encoder(dtype="bf16", B=2, T=64, ragged=True, width=16)
    d = si.draw(w)
    saved, lens = O.encoder_fwd(w.layers, d.x, d.lengths, d.params)
    grads, dx, _ = O.encoder_bwd(w.layers, d.g, lens, d.params, saved)
    t = dict(layers=w.layers, dtype="bf16", x=d.x, lengths=d.lengths, params=d.params, g=d.g,
             ys=[t16(S["y"], "bf16") for S in saved], gate_extra=[None] * len(w.layers), dx=t16(dx, "bf16"),
             grads=[{k: torch.tensor(v, dtype=torch.float32) for k, v in G.items() if k != "dx"} for G in grads])
    out = U.end_to_end_task(t)
    assert max(out["y"]) <= 1.0 and out["dx"] <= 1.0 and out["hard"] == 0
    assert all(e <= 1e-3 for rows in out["grads"] for _, e in rows)
    ctl = U.storage_control_task(dict(layers=w.layers, dtype="bf16", x=d.x, lengths=d.lengths, params=d.params, g=d.g))
    assert len(ctl["y"]) == len(w.layers) and ctl["y"][0] <= 1.0
    assert ctl["y"][-1] >= ctl["y"][0] * 0.5           # rounding error does not shrink with depth
