"""Pins for the whole-forward oracle: brute force on tiny models, the sharding
invariant of Eq. 1-2, incremental decoding, a closed form, and the library
model the paper's prototype is built on (Sec. 4: HF Transformers Llama)."""
import numpy as np
import pytest

import tpi_synth as S
from oracle import brute
from oracle.llama_oracle import LlamaOracle
from tests.helpers import TINY, make_oracle, oracle_cfg, rel_l2, weight_fn


def test_brute_force_agrees_on_tiny_models():
    for shape in (TINY, TINY.with_(n_heads=2, n_kv_heads=2, head_dim=16, seed=8),
                  TINY.with_(n_layers=1, n_heads=4, n_kv_heads=1, seed=9, rope_base=500000.0)):
        orc = make_oracle(shape)
        toks = S.prompt_tokens(shape, 6)
        got = orc.forward(toks, all_logits=True)
        w = weight_fn(shape)
        cfg = dict(n_layers=shape.n_layers, hidden=shape.hidden, n_heads=shape.n_heads,
                   n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, ffn=shape.ffn,
                   vocab=shape.vocab, rms_eps=shape.rms_eps, rope_base=shape.rope_base)
        want = np.array(brute.forward_tokens(cfg, lambda l, t: w(l, t).tolist(), toks.tolist()))
        assert rel_l2(got, want) < 1e-13


@pytest.mark.parametrize("n_shards", [1, 2, 4])
def test_sharded_sum_equals_unsharded_layer(n_shards):
    shape = S.CONFIGS["C1"]
    a, b = make_oracle(shape), make_oracle(shape)
    toks = S.prompt_tokens(shape)
    la = a.forward(toks)
    lb = b.forward(toks, n_shards=n_shards)
    assert rel_l2(lb, la) < 1e-12
    for l in range(shape.n_layers):
        for k in ("attn", "ffn"):
            assert rel_l2(b.taps[(l, k)], a.taps[(l, k)]) < 1e-12
    # the caches are the same object whichever way the heads were split
    assert rel_l2(np.stack(b.cache.K), np.stack(a.cache.K)) < 1e-13
    # one more decoded position through the sharded path
    assert rel_l2(b.forward([5], n_shards=n_shards), a.forward([5])) < 1e-12


def test_token_ids_do_not_depend_on_n():
    shape = S.CONFIGS["C1"]
    toks = S.prompt_tokens(shape)
    ref, _ = make_oracle(shape).greedy(toks, 8)
    for n in (1, 2, 4):
        got, _ = make_oracle(shape).greedy(toks, 8, n_shards=n)
        assert (got == ref).all()


def test_gqa_sharding_invariant():
    shape = TINY.with_(n_heads=8, n_kv_heads=4, head_dim=4, ffn=48)
    toks = S.prompt_tokens(shape, 7)
    ref = make_oracle(shape).forward(toks)
    for n in (2, 4):
        assert rel_l2(make_oracle(shape).forward(toks, n_shards=n), ref) < 1e-12
    with pytest.raises(ValueError):
        make_oracle(shape).forward(toks, n_shards=8)          # 8 does not divide 4 kv heads


def test_incremental_decoding_equals_longer_prefill():
    shape = S.CONFIGS["C1"]
    toks = S.prompt_tokens(shape, 12)
    full = make_oracle(shape).forward(toks, all_logits=True)
    inc = make_oracle(shape)
    inc.forward(toks[:7])
    for t in range(7, 12):
        lg = inc.forward(toks[t:t + 1])
        assert rel_l2(lg, full[t]) < 1e-12
    assert inc.cache.length == 12 and inc.cache.K[0].shape == (shape.n_kv_heads, 12, shape.head_dim)


def test_closed_form_when_output_projections_vanish():
    shape = TINY
    base = weight_fn(shape)

    def w(l, t):
        m = base(l, t)
        return np.zeros_like(m) if t in (S.WO, S.WDOWN) else m
    orc = LlamaOracle(oracle_cfg(shape), w)
    toks = S.prompt_tokens(shape, 4)
    x = base(0, S.EMB)[toks[-1]]
    xn = x / np.sqrt((x * x).mean() + shape.rms_eps) * base(0, S.FINAL_NORM)
    assert rel_l2(orc.forward(toks), base(0, S.HEAD) @ xn) < 1e-14


def test_kv_rounding_switch():
    shape = S.CONFIGS["C1"]
    toks = S.prompt_tokens(shape)
    exact = make_oracle(shape, "none")
    rounded = make_oracle(shape, "bf16")
    le, lr = exact.forward(toks), rounded.forward(toks)
    K = rounded.cache.K[0]
    u = K.astype(np.float32).view(np.uint32)
    assert (K.astype(np.float32) == K).all() and (u & 0xFFFF == 0).all()    # values sit on the bf16 grid
    assert 1e-6 < rel_l2(lr, le) < 1e-2


def test_matches_transformers_llama():
    """The prototype in the paper is HF Transformers' Llama; a randomly initialised
    instance loaded with the generated weights is the paper's own definition."""
    torch = pytest.importorskip("torch")
    tr = pytest.importorskip("transformers")
    for shape in (S.CONFIGS["C1"], TINY.with_(n_heads=8, n_kv_heads=2, head_dim=4, rope_base=500000.0)):
        cfg = tr.LlamaConfig(vocab_size=shape.vocab, hidden_size=shape.hidden, intermediate_size=shape.ffn,
                             num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_heads,
                             num_key_value_heads=shape.n_kv_heads, head_dim=shape.head_dim,
                             rms_norm_eps=shape.rms_eps, max_position_embeddings=64,
                             tie_word_embeddings=False, attention_bias=False, mlp_bias=False,
                             rope_parameters={"rope_theta": shape.rope_base, "rope_type": "default"},
                             attn_implementation="eager")
        model = tr.LlamaForCausalLM(cfg).double().eval()
        w = weight_fn(shape)
        sd = {"model.embed_tokens.weight": w(0, S.EMB), "lm_head.weight": w(0, S.HEAD),
              "model.norm.weight": w(0, S.FINAL_NORM)}
        names = {S.ATTN_NORM: "input_layernorm", S.WQ: "self_attn.q_proj", S.WK: "self_attn.k_proj",
                 S.WV: "self_attn.v_proj", S.WO: "self_attn.o_proj", S.FFN_NORM: "post_attention_layernorm",
                 S.WGATE: "mlp.gate_proj", S.WUP: "mlp.up_proj", S.WDOWN: "mlp.down_proj"}
        for l in range(shape.n_layers):
            for tid, nm in names.items():
                sd[f"model.layers.{l}.{nm}.weight"] = w(l, tid)
        missing = model.load_state_dict({k: torch.from_numpy(np.ascontiguousarray(v)) for k, v in sd.items()},
                                        strict=False)
        assert not [m for m in missing.missing_keys if "rotary" not in m] and not missing.unexpected_keys
        toks = S.prompt_tokens(shape, 12)
        with torch.no_grad():
            want = model(torch.from_numpy(toks.astype(np.int64))[None]).logits[0].numpy()
        got = make_oracle(shape, "none").forward(toks, all_logits=True)
        # the library builds its rotary tables in float32, so agreement is ~1e-7, not 1e-15
        assert rel_l2(got, want) < 1e-5
        assert (got.argmax(-1) == want.argmax(-1)).all()


def test_heterogeneous_partition_equals_unsharded_and_the_uniform_one():
    """Sec. 3.1: device i takes a proportion p_i of the heads and of the FFN columns; whatever the proportions,
    the sum of the devices' partial results is the unsharded layer (the paper's identity with single-server
    inference), and the uniform proportions reproduce the default split exactly."""
    shape = TINY.with_(n_heads=8, n_kv_heads=4, head_dim=4, ffn=48)
    toks = S.prompt_tokens(shape, 7)
    ref = make_oracle(shape)
    want = ref.forward(toks)
    for n, part in ((2, ([3, 1], [40, 8])), (3, ([2, 1, 1], [24, 16, 8])), (4, ([1, 1, 1, 1], [8, 8, 8, 24]))):
        o = make_oracle(shape)
        assert rel_l2(o.forward(toks, n_shards=n, partition=part), want) < 1e-12
        for l in range(shape.n_layers):
            assert rel_l2(o.taps[(l, "ffn")], ref.taps[(l, "ffn")]) < 1e-12
        assert rel_l2(np.stack(o.cache.K), np.stack(ref.cache.K)) < 1e-13
    u, v = make_oracle(shape), make_oracle(shape)
    assert np.array_equal(u.forward(toks, n_shards=2), v.forward(toks, n_shards=2, partition=([2, 2], [24, 24])))
    for bad in (([4, 1], [24, 24]), ([2, 2], [24, 16]), ([4, 0], [24, 24]), ([2, 2, 0], [24, 24])):
        with pytest.raises(ValueError):
            make_oracle(shape).forward(toks, n_shards=2, partition=bad)
