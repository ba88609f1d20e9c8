"""Quantised frozen base with 16-bit adapters (the paper's Sec. 5 variant): the library's dequantisation bit for bit
against the oracle's, and a decoder forward whose seven projections per block read 8-bit base weights."""
import numpy as np
import pytest
import torch

import moin_inputs as mi
import oracle
import paper_2410_09687_b200 as moin
from gpu_util import DEV, REL_FRO

pytestmark = pytest.mark.gpu


def quantise(W: torch.Tensor):
    """Test-side quantiser (torch): per-row scale max|w| / 448, nearest 8-bit float code."""
    scale = (W.float().abs().amax(dim=1) / 448.0).clamp_min(1e-12)
    codes = (W.float() / scale[:, None]).to(torch.float8_e4m3fn).view(torch.uint8)
    return codes.contiguous(), scale.contiguous()


@pytest.mark.parametrize("shape", [(1, 16), (7, 48), (256, 2048), (1000, 5632)])
def test_dequantisation_bit_for_bit(shape):
    rng = np.random.default_rng(shape[0])
    codes = rng.integers(0, 256, size=shape).astype(np.uint8)
    codes[(codes & 0x7F) == 0x7F] = 0x01                      # every code but the two NaNs, subnormals and -0 included
    scale = np.exp(rng.uniform(-8, 2, size=shape[0])).astype(np.float32)
    got = moin.dequant_fp8(torch.from_numpy(codes).to(DEV), torch.from_numpy(scale).to(DEV))
    torch.cuda.synchronize()
    assert np.array_equal(mi.bf16_bits(got.cpu()), oracle.dequant_fp8(codes, scale))


def test_argument_errors():
    c = torch.zeros(4, 24, dtype=torch.uint8, device=DEV)
    with pytest.raises(moin.MoinError, match="BAD_SHAPE"):
        moin.dequant_fp8(c, torch.ones(4, device=DEV))


def test_decoder_on_a_quantised_base():
    cfg = mi.DecoderConfig(n_layers=2, hidden=256, n_heads=4, n_kv_heads=2, head_dim=64, ffn=512, vocab=1000,
                           E=6, r=16, scale=2.0)
    model = mi.decoder_model(cfg, seed=9, missing=(2,))
    order = oracle.PROJ_ORDER
    W8, Ws, Wdq = [], [], []
    for l in range(cfg.n_layers):
        q = {p: quantise(model.W[l][p]) for p in order}
        W8.append({p: q[p][0].to(DEV) for p in order})
        Ws.append({p: q[p][1].to(DEV) for p in order})
        Wdq.append({p: oracle.dequant_fp8(q[p][0].numpy(), q[p][1].numpy()) for p in order})
    # quantisation is not a no-op here (else the test would not see a base that ignores the codes)
    d = mi.bf16_to_f64(model.W[0]["q"]) - mi.bf16_to_f64(torch.from_numpy(Wdq[0]["q"].view(np.int16)).view(torch.bfloat16))
    assert np.linalg.norm(d) / np.linalg.norm(mi.bf16_to_f64(model.W[0]["q"])) > 1e-2
    pools = [{p: moin.Pool(model.pools[l][p].A.to(DEV), model.pools[l][p].B.to(DEV),
                           model.pools[l][p].slot_of_expert.to(DEV)) for p in order} for l in range(cfg.n_layers)]
    gm = moin.DecoderModel(cfg, model.embed.to(DEV), model.lm_head.to(DEV), model.final_norm.to(DEV),
                           [t.to(DEV) for t in model.attn_norm], [t.to(DEV) for t in model.mlp_norm],
                           [{} for _ in range(cfg.n_layers)], pools, cfg.E, cfg.scale, W8=W8, W_scale=Ws)
    orc = oracle.DecoderOracle(cfg, {
        "embed": mi.bf16_bits(model.embed), "lm_head": mi.bf16_bits(model.lm_head), "final_norm": mi.bf16_bits(model.final_norm),
        "attn_norm": [mi.bf16_bits(t) for t in model.attn_norm], "mlp_norm": [mi.bf16_bits(t) for t in model.mlp_norm],
        "W": Wdq, "A": [{p: mi.bf16_bits(model.pools[l][p].A) for p in order} for l in range(cfg.n_layers)],
        "B": [{p: mi.bf16_bits(model.pools[l][p].B) for p in order} for l in range(cfg.n_layers)],
        "slot_of_expert": model.pools[0]["q"].slot_of_expert.numpy()})
    for lengths, experts in (([70, 1, 129, 33], [0, 2, 3, -1]), ([200, 130], [1, 4])):   # short segments / long runs
        batch = mi.decoder_batch(cfg, lengths, seed=9, req_expert=experts)
        logits = moin.decoder_forward(gm, batch.tokens.to(DEV), batch.cu_seqlens.to(DEV), batch.req_expert.to(DEV), max(lengths))
        torch.cuda.synchronize()
        args = (batch.tokens.numpy(), batch.cu_seqlens.numpy(), batch.req_expert.numpy())
        rounded = orc.forward(*args, round_storage=True)["logits"]
        exact = orc.forward(*args)["logits"]
        got = logits.double().cpu().numpy()
        e_r = np.linalg.norm(got - rounded) / np.linalg.norm(rounded)
        e_x = np.linalg.norm(got - exact) / np.linalg.norm(exact)
        print(f"quantised base, lengths {lengths}: logits vs storage-rounded oracle {e_r:.2e}, vs fp64 oracle {e_x:.2e}")
        assert e_r <= REL_FRO * np.sqrt(cfg.n_layers + 1) and e_x <= 2 * REL_FRO * np.sqrt(cfg.n_layers + 1)
    assert moin.device_status()["timeout_flag"] == 0
