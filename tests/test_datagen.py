import numpy as np
import torch

import datagen


def test_streams_are_deterministic_and_distinct():
    cfg = datagen.CONFIGS["tiny"]
    a = datagen.layer_weights(cfg, 3)
    b = datagen.layer_weights(cfg, 3)
    c = datagen.layer_weights(cfg, 4)
    for k in a:
        assert torch.equal(a[k], b[k])
    assert not torch.equal(a["wq"], c["wq"])
    assert not torch.equal(a["w_gate"], a["w_up"])
    assert a["wq"].shape == (256, 256) and a["w_down"].shape == (256, 688)
    assert a["wk"].shape == (128, 256) and a["wq"].dtype == torch.float32


def test_normal_moments_and_out_proj_scale():
    z = datagen.standard_normal(datagen.stream_key(9, 0, 0), 1 << 18)
    assert abs(float(z.mean())) < 0.01 and abs(float(z.std()) - 1.0) < 0.01
    assert abs(float((z ** 4).mean()) - 3.0) < 0.1           # kurtosis of a normal
    cfg = datagen.CONFIGS["mini8b"]
    w = datagen.layer_weights(cfg, 0)
    assert w["wq"].dtype == torch.bfloat16
    s_in, s_out = float(w["wq"].float().std()), float(w["wo"].float().std())
    assert abs(s_in - 0.02) < 1e-3
    assert abs(s_out - 0.02 / np.sqrt(2 * cfg.L)) < 1e-3


def test_token_ids_in_range():
    cfg = datagen.CONFIGS["8b"]
    t = datagen.token_ids(cfg, 4096)
    assert t.dtype == torch.int32 and int(t.min()) >= 0 and int(t.max()) < cfg.vocab
    assert len(torch.unique(t)) > 3900
    assert torch.equal(t, datagen.token_ids(cfg, 4096))
