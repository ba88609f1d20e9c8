"""Pins for the oracle's decoder forward (Sec. 4: the base model has the Llama-2 architecture;
Sec. 3.2/3.3: the request's adapter on every linear layer of every block).

External pin: the `transformers` Llama implementation run in float64 on the same random
weights - for the base model (all requests without an adapter) and, through the LoRA merge
identity W + s W_b W_a, for a request routed to an expert.  Structural pins: a request gives
the same result alone and inside a batch; block-by-block feeding reproduces the full forward.
"""
import numpy as np
import pytest
import torch

import moin_inputs as mi
import oracle

CFG = mi.DecoderConfig(n_layers=2, hidden=64, n_heads=4, n_kv_heads=2, head_dim=16, ffn=128, vocab=97,
                       E=4, r=8, scale=2.0)
# transformers builds its rotary cos/sin tables in float32 even for a float64 model, which moves
# logits by ~1e-8..1e-7 here; a structural mistake (pairing, head mapping, norm, mask) moves them by ~1e-2.
HF_ATOL = 1e-6
HF_NAMES = {"q": "self_attn.q_proj", "k": "self_attn.k_proj", "v": "self_attn.v_proj", "o": "self_attn.o_proj",
            "gate": "mlp.gate_proj", "up": "mlp.up_proj", "down": "mlp.down_proj"}


def oracle_weights(model: mi.DecoderModel, with_adapters=True) -> dict:
    nl = model.cfg.n_layers
    w = {"embed": mi.bf16_bits(model.embed), "lm_head": mi.bf16_bits(model.lm_head),
         "final_norm": mi.bf16_bits(model.final_norm),
         "attn_norm": [mi.bf16_bits(t) for t in model.attn_norm],
         "mlp_norm": [mi.bf16_bits(t) for t in model.mlp_norm],
         "W": [{p: mi.bf16_bits(model.W[l][p]) for p in oracle.PROJ_ORDER} for l in range(nl)],
         "slot_of_expert": model.pools[0]["q"].slot_of_expert.cpu().numpy()}
    if with_adapters:
        w["A"] = [{p: mi.bf16_bits(model.pools[l][p].A) for p in oracle.PROJ_ORDER} for l in range(nl)]
        w["B"] = [{p: mi.bf16_bits(model.pools[l][p].B) for p in oracle.PROJ_ORDER} for l in range(nl)]
    return w


def hf_llama(model: mi.DecoderModel, merged_expert=None):
    from transformers import LlamaConfig, LlamaForCausalLM
    c = model.cfg
    hf = LlamaForCausalLM(LlamaConfig(
        vocab_size=c.vocab, hidden_size=c.hidden, intermediate_size=c.ffn, num_hidden_layers=c.n_layers,
        num_attention_heads=c.n_heads, num_key_value_heads=c.n_kv_heads, head_dim=c.head_dim,
        rms_norm_eps=c.rms_eps, rope_theta=c.rope_base, attention_bias=False, mlp_bias=False,
        tie_word_embeddings=False, max_position_embeddings=512)).to(torch.float64).eval()
    sd = {"model.embed_tokens.weight": model.embed, "lm_head.weight": model.lm_head,
          "model.norm.weight": model.final_norm}
    for l in range(c.n_layers):
        sd[f"model.layers.{l}.input_layernorm.weight"] = model.attn_norm[l]
        sd[f"model.layers.{l}.post_attention_layernorm.weight"] = model.mlp_norm[l]
        for p, hn in HF_NAMES.items():
            Wm = model.W[l][p].to(torch.float64)
            if merged_expert is not None:
                pool = model.pools[l][p]
                s = int(pool.slot_of_expert[merged_expert])
                if s >= 0:
                    Wm = Wm + c.scale * (pool.B[s].to(torch.float64) @ pool.A[s].to(torch.float64))
            sd[f"model.layers.{l}.{hn}.weight"] = Wm
    missing, unexpected = hf.load_state_dict({k: v.to(torch.float64) for k, v in sd.items()}, strict=False)
    assert not [m for m in missing if "rotary" not in m] and not unexpected
    return hf


@pytest.fixture(scope="module")
def setup():
    model = mi.decoder_model(CFG, seed=4, missing=(2,))
    batch = mi.decoder_batch(CFG, [9, 1, 17, 5], seed=4, req_expert=[0, 2, 3, -1])
    return model, batch, oracle.DecoderOracle(CFG, oracle_weights(model))


def test_base_model_matches_transformers_llama_fp64(setup):
    model, batch, orc = setup
    hf = hf_llama(model)
    cu = batch.cu_seqlens.numpy()
    out = orc.forward(batch.tokens.numpy(), cu, np.full(batch.R, -1, np.int32))["logits"]
    for r in range(batch.R):
        ids = batch.tokens[cu[r]:cu[r + 1]].long()[None]
        with torch.no_grad():
            ref = hf(ids).logits[0].numpy()
        np.testing.assert_allclose(out[cu[r]:cu[r + 1]], ref, rtol=0, atol=HF_ATOL)
    # experts without an adapter (2) and no expert (-1) are the base model too
    alt = orc.forward(batch.tokens.numpy(), cu, np.array([2, -1, 2, -1], np.int32))["logits"]
    assert np.array_equal(alt, out)


def test_routed_request_matches_transformers_llama_with_merged_adapter(setup):
    model, batch, orc = setup
    cu = batch.cu_seqlens.numpy()
    out = orc.forward(batch.tokens.numpy(), cu, batch.req_expert.numpy())["logits"]
    base = orc.forward(batch.tokens.numpy(), cu, np.full(batch.R, -1, np.int32))["logits"]
    for r, e in enumerate(batch.req_expert.numpy()):
        hf = hf_llama(model, merged_expert=None if e < 0 else int(e))
        ids = batch.tokens[cu[r]:cu[r + 1]].long()[None]
        with torch.no_grad():
            ref = hf(ids).logits[0].numpy()
        np.testing.assert_allclose(out[cu[r]:cu[r + 1]], ref, rtol=0, atol=HF_ATOL)
    # the adapter must matter for routed requests 0 and 2, and only for them
    assert np.abs(out[cu[0]:cu[1]] - base[cu[0]:cu[1]]).max() > 1e-3
    assert np.array_equal(out[cu[1]:cu[2]], base[cu[1]:cu[2]])
    assert np.array_equal(out[cu[3]:cu[4]], base[cu[3]:cu[4]])


def test_request_alone_equals_request_in_batch(setup):
    model, batch, orc = setup
    cu = batch.cu_seqlens.numpy()
    full = orc.forward(batch.tokens.numpy(), cu, batch.req_expert.numpy())["logits"]
    for r in range(batch.R):
        one = orc.forward(batch.tokens.numpy()[cu[r]:cu[r + 1]], np.array([0, cu[r + 1] - cu[r]]),
                          batch.req_expert.numpy()[r:r + 1])["logits"]
        assert np.array_equal(one, full[cu[r]:cu[r + 1]])


def test_block_by_block_feeding_reproduces_full_forward(setup):
    model, batch, orc = setup
    args = (batch.tokens.numpy(), batch.cu_seqlens.numpy(), batch.req_expert.numpy())
    full = orc.forward(*args, want_hidden=True)
    h0 = orc.forward(*args, layer_begin=0, layer_end=0, want_hidden=True, want_logits=False)["hidden"]
    assert np.array_equal(h0, mi.bf16_to_f64(model.embed)[batch.tokens.numpy()])
    h1 = orc.forward(*args, layer_begin=0, layer_end=1, want_hidden=True, want_logits=False)["hidden"]
    h2 = orc.forward(*args, layer_begin=1, layer_end=2, hidden_in=h1, want_hidden=True)
    assert np.array_equal(h2["hidden"], full["hidden"])
    assert np.array_equal(h2["logits"], full["logits"])


def test_storage_rounded_variant_stays_close_and_is_bf16(setup):
    model, batch, orc = setup
    args = (batch.tokens.numpy(), batch.cu_seqlens.numpy(), batch.req_expert.numpy())
    exact = orc.forward(*args)["logits"]
    rounded = orc.forward(*args, round_storage=True)["logits"]
    as_bf16 = torch.from_numpy(rounded).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(as_bf16, rounded)            # every logit is a bf16 value
    rel = np.linalg.norm(rounded - exact) / np.linalg.norm(exact)
    assert 0 < rel < 2e-2
