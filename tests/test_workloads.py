"""The seeded input generators: deterministic, right shapes, no dependence on chunking."""

import torch

import workloads as WL


def test_generators_are_deterministic_and_typed():
    a = WL.make_weight(16, 32, "bf16", seed=3, layer_index=1)
    b = WL.make_weight(16, 32, "bf16", seed=3, layer_index=1)
    c = WL.make_weight(16, 32, "bf16", seed=3, layer_index=2)
    assert a.dtype == torch.bfloat16 and torch.equal(a, b) and not torch.equal(a, c)
    assert 0.01 < float(a.float().std()) < 0.03
    x = WL.make_activations(WL.TOKEN_CHUNK + 100, 64, "f32", "student_t4", 0.05, 0, 20.0, 9, 0)
    y = WL.make_activations(WL.TOKEN_CHUNK, 64, "f32", "student_t4", 0.05, 0, 20.0, 9, 0)
    assert torch.equal(x[: WL.TOKEN_CHUNK], y)
    ch = WL.outlier_channels(64, 0.05, 0, 9, 0)
    assert len(ch) == 3
    norms = x.pow(2).mean(0).sqrt()
    others = torch.ones(64, dtype=torch.bool)
    others[ch] = False
    assert float(norms[ch].min()) > 5 * float(norms[others].max())


def test_config_table_matches_the_named_shapes():
    c = WL.CONFIGS["llama2_7b"]
    assert sorted((L.c, L.b) for L in c.layers) == sorted(
        [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)])
    assert c.a == 262144 and c.B == 128 and c.p == 0.5 and c.dtype == "bf16"
    t = WL.CONFIGS["tiny"]
    assert (t.layers[0].c, t.layers[0].b, t.a, t.B, t.outlier_count) == (256, 256, 2048, 64, 4)
    o = WL.CONFIGS["opt125m"]
    assert (o.n, o.m, o.B, o.dtype) == (2, 4, 128, "f32")
    l3 = WL.CONFIGS["llama3_8b"]
    assert (l3.n, l3.m, l3.B) == (4, 8, 256)
