"""Decoder forward on the GPU against the oracle (Llama-architecture blocks whose projections are routed
LoRA layers).  Gate: block by block with the oracle's own block input (teacher forcing), and end to end
against the oracle variant that rounds to bf16 where the library stores bf16; the distance to the pure
fp64 oracle is printed."""
import numpy as np
import pytest
import torch

import moin_inputs as mi
import oracle
import paper_2410_09687_b200 as moin
from gpu_util import DEV, REL_FRO

pytestmark = pytest.mark.gpu

CFG = mi.DecoderConfig(n_layers=3, hidden=256, n_heads=4, n_kv_heads=2, head_dim=64, ffn=512, vocab=1000,
                       E=6, r=16, scale=2.0)


def oracle_weights(model):
    nl = model.cfg.n_layers
    return {"embed": mi.bf16_bits(model.embed), "lm_head": mi.bf16_bits(model.lm_head),
            "final_norm": mi.bf16_bits(model.final_norm),
            "attn_norm": [mi.bf16_bits(t) for t in model.attn_norm],
            "mlp_norm": [mi.bf16_bits(t) for t in model.mlp_norm],
            "W": [{p: mi.bf16_bits(model.W[l][p]) for p in oracle.PROJ_ORDER} for l in range(nl)],
            "A": [{p: mi.bf16_bits(model.pools[l][p].A) for p in oracle.PROJ_ORDER} for l in range(nl)],
            "B": [{p: mi.bf16_bits(model.pools[l][p].B) for p in oracle.PROJ_ORDER} for l in range(nl)],
            "slot_of_expert": model.pools[0]["q"].slot_of_expert.cpu().numpy()}


def gpu_model(model):
    nl = model.cfg.n_layers
    pools = [{p: moin.Pool(model.pools[l][p].A.to(DEV), model.pools[l][p].B.to(DEV),
                           model.pools[l][p].slot_of_expert.to(DEV)) for p in oracle.PROJ_ORDER} for l in range(nl)]
    W = [{p: model.W[l][p].to(DEV) for p in oracle.PROJ_ORDER} for l in range(nl)]
    return moin.DecoderModel(model.cfg, model.embed.to(DEV), model.lm_head.to(DEV), model.final_norm.to(DEV),
                             [t.to(DEV) for t in model.attn_norm], [t.to(DEV) for t in model.mlp_norm], W, pools,
                             model.cfg.E, model.cfg.scale)


def rel(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


@pytest.fixture(scope="module")
def setup():
    model = mi.decoder_model(CFG, seed=4, missing=(2,))
    return model, gpu_model(model), oracle.DecoderOracle(CFG, oracle_weights(model))


@pytest.mark.parametrize("lengths,experts", [([70, 1, 129, 33, 64], [0, 2, 3, -1, 5]),      # short requests: segments
                                             ([200, 130, 257], [1, 1, 4]),                  # long runs: tiles
                                             ([3, 530, 260], [5, 2, 0])])     # attention items beyond 256 keys
def test_decoder_end_to_end_and_block_by_block(setup, lengths, experts):
    model, gm, orc = setup
    batch = mi.decoder_batch(CFG, lengths, seed=4, req_expert=experts)
    tok, cu, re_ = batch.tokens.to(DEV), batch.cu_seqlens.to(DEV), batch.req_expert.to(DEV)
    args = (batch.tokens.numpy(), batch.cu_seqlens.numpy(), batch.req_expert.numpy())
    hid = torch.empty(batch.T, CFG.hidden, dtype=torch.float32, device=DEV)
    # Gate 1 - block by block: the GPU block gets the oracle's (storage-rounded) block input, and the
    # block's contribution to the residual stream must meet the layer tolerance.
    h_in = orc.forward(*args, layer_begin=0, layer_end=0, want_hidden=True, want_logits=False)["hidden"]
    for l in range(CFG.n_layers):
        ref = orc.forward(*args, layer_begin=l, layer_end=l + 1, round_storage=True, hidden_in=h_in,
                          want_hidden=True, want_logits=False)["hidden"]
        hin_gpu = torch.from_numpy(h_in).to(torch.float32).to(DEV)
        moin.decoder_forward(gm, tok, cu, re_, max(lengths), logits_mode=moin.LOGITS_NONE, hidden_in=hin_gpu,
                             hidden_out=hid, layer_begin=l, layer_end=l + 1)
        torch.cuda.synchronize()
        d = hid.double().cpu().numpy() - hin_gpu.double().cpu().numpy()
        e_blk = rel(d, ref - h_in)
        print(f"block {l}: rel Frobenius of the block's residual update {e_blk:.2e}")
        assert e_blk <= REL_FRO, f"block {l}"
        h_in = ref
    # Gate 2 - end to end: rounding differences of every block add up like a random walk, so the
    # logits get the layer tolerance times sqrt(blocks + 1) against the storage-rounded oracle; the
    # distance to the pure fp64 oracle is printed.
    logits = moin.decoder_forward(gm, tok, cu, re_, max(lengths), hidden_out=hid)
    torch.cuda.synchronize()
    got = logits.to(torch.float64).cpu().numpy()
    assert np.isfinite(got).all()
    exact = orc.forward(*args)["logits"]
    rounded = orc.forward(*args, round_storage=True, want_hidden=True)
    e_exact, e_round = rel(got, exact), rel(got, rounded["logits"])
    print(f"logits rel Frobenius: vs fp64 oracle {e_exact:.2e}, vs storage-rounded oracle {e_round:.2e}")
    tol = REL_FRO * np.sqrt(CFG.n_layers + 1)
    assert e_round <= tol and e_exact <= 2 * tol
    assert rel(hid.double().cpu().numpy(), rounded["hidden"]) <= tol


def test_decoder_last_token_logits_and_request_independence(setup):
    model, gm, orc = setup
    lengths, experts = [40, 7, 90], [3, 0, -1]
    batch = mi.decoder_batch(CFG, lengths, seed=5, req_expert=experts)
    tok, cu, re_ = batch.tokens.to(DEV), batch.cu_seqlens.to(DEV), batch.req_expert.to(DEV)
    full = moin.decoder_forward(gm, tok, cu, re_, 90)
    last = moin.decoder_forward(gm, tok, cu, re_, 90, logits_mode=moin.LOGITS_LAST)
    torch.cuda.synchronize()
    cuh = batch.cu_seqlens.numpy()
    assert torch.equal(last, full[torch.from_numpy(cuh[1:] - 1).long().to(DEV)])
    # a request alone gives the same logits as inside the batch (introvert experts)
    for r in range(3):
        one = moin.decoder_forward(gm, tok[cuh[r]:cuh[r + 1]].contiguous(),
                                   torch.tensor([0, lengths[r]], dtype=torch.int32, device=DEV),
                                   re_[r:r + 1].contiguous(), lengths[r])
        ref = full[cuh[r]:cuh[r + 1]].double()
        assert float((one.double() - ref).norm() / ref.norm()) <= REL_FRO


def test_decoder_per_token_experts(setup):
    """One expert per token (the paper's future-work variant, Sec. 5).  Ids constant inside each request reproduce
    the per-request forward bit for bit; mixed ids are checked block by block and end to end against the oracle."""
    model, gm, orc = setup
    lengths, experts = [70, 1, 129, 33, 64], [0, 2, 3, -1, 5]
    batch = mi.decoder_batch(CFG, lengths, seed=8, req_expert=experts)
    tok, cu, re_ = batch.tokens.to(DEV), batch.cu_seqlens.to(DEV), batch.req_expert.to(DEV)
    te_const = torch.repeat_interleave(batch.req_expert, torch.tensor(lengths)).to(torch.int32).to(DEV)
    a = moin.decoder_forward(gm, tok, cu, re_, max(lengths))
    b = moin.decoder_forward(gm, tok, cu, None, max(lengths), token_expert=te_const)
    torch.cuda.synchronize()
    # (the per-token call lets the plan pick its mode from the grouped ids, the per-request call from the request
    # lengths: same values, not necessarily the same kernels)
    assert float((a.double() - b.double()).norm() / a.double().norm()) <= REL_FRO
    rng = np.random.default_rng(3)
    for flavour in ("mixed", "runs"):
        if flavour == "mixed":      # ids change from token to token: short segments
            te = rng.integers(-1, CFG.E, size=batch.T).astype(np.int32)
        else:                       # ids change every ~50 tokens, across request borders: long runs
            te = np.repeat(rng.integers(-1, CFG.E, size=batch.T // 50 + 1), 50)[:batch.T].astype(np.int32)
        te_d = torch.from_numpy(te).to(DEV)
        args = (batch.tokens.numpy(), batch.cu_seqlens.numpy(), None)
        hid = torch.empty(batch.T, CFG.hidden, dtype=torch.float32, device=DEV)
        h_in = orc.forward(*args, layer_begin=0, layer_end=0, want_hidden=True, want_logits=False)["hidden"]
        for l in range(CFG.n_layers):
            ref = orc.forward(*args, layer_begin=l, layer_end=l + 1, round_storage=True, hidden_in=h_in,
                              want_hidden=True, want_logits=False, token_expert=te)["hidden"]
            hin_gpu = torch.from_numpy(h_in).to(torch.float32).to(DEV)
            moin.decoder_forward(gm, tok, cu, None, max(lengths), logits_mode=moin.LOGITS_NONE, hidden_in=hin_gpu,
                                 hidden_out=hid, layer_begin=l, layer_end=l + 1, token_expert=te_d)
            torch.cuda.synchronize()
            d = hid.double().cpu().numpy() - hin_gpu.double().cpu().numpy()
            assert rel(d, ref - h_in) <= REL_FRO, f"{flavour} block {l}"
            h_in = ref
        logits = moin.decoder_forward(gm, tok, cu, None, max(lengths), token_expert=te_d)
        torch.cuda.synchronize()
        rounded = orc.forward(*args, round_storage=True, token_expert=te)["logits"]
        e = rel(logits.double().cpu().numpy(), rounded)
        print(f"per-token experts ({flavour}): logits vs storage-rounded oracle {e:.2e}")
        assert e <= REL_FRO * np.sqrt(CFG.n_layers + 1)
        # per-token ids are not per-request ids in disguise: forcing each request's first id changes the result
        first = torch.repeat_interleave(te_d[cu[:-1].long()], torch.tensor(lengths, device=DEV)).to(torch.int32)
        other = moin.decoder_forward(gm, tok, cu, None, max(lengths), token_expert=first)
        assert float((other.double() - logits.double()).norm() / logits.double().norm()) > 10 * REL_FRO
    assert moin.device_status()["timeout_flag"] == 0


@pytest.mark.parametrize("lengths,experts", [([130, 1, 64, 70], [3, -1, 9, 3]),            # long runs -> tile mode
                                             ([5, 9, 1, 12, 7, 3, 8, 2], [1, 2, 3, 4, 5, 6, 7, 1])])  # decode-like
def test_decoder_full_width_blocks(lengths, experts):
    """TinyLlama-width blocks (hidden 2048, 32/4 heads, SwiGLU 5632, vocab 32000, rank 64): every block is
    checked with the oracle's own block input, and the logits of the last block's output too."""
    cfg = mi.DecoderConfig(n_layers=2, E=16, r=64)
    model = mi.decoder_model(cfg, seed=6, missing=(9,))
    gm, orc = gpu_model(model), oracle.DecoderOracle(cfg, oracle_weights(model))
    batch = mi.decoder_batch(cfg, lengths, seed=6, req_expert=experts)
    tok, cu, re_ = batch.tokens.to(DEV), batch.cu_seqlens.to(DEV), batch.req_expert.to(DEV)
    args = (batch.tokens.numpy(), batch.cu_seqlens.numpy(), batch.req_expert.numpy())
    hid = torch.empty(batch.T, cfg.hidden, dtype=torch.float32, device=DEV)
    h_in = orc.forward(*args, layer_begin=0, layer_end=0, want_hidden=True, want_logits=False)["hidden"]
    for l in range(cfg.n_layers):
        last = l == cfg.n_layers - 1
        ref = orc.forward(*args, layer_begin=l, layer_end=l + 1, round_storage=True, hidden_in=h_in,
                          want_hidden=True, want_logits=last)
        exact = orc.forward(*args, layer_begin=l, layer_end=l + 1, round_storage=False, hidden_in=h_in,
                            want_hidden=True, want_logits=False)["hidden"]
        hin_gpu = torch.from_numpy(h_in).to(torch.float32).to(DEV)
        logits = moin.decoder_forward(gm, tok, cu, re_, max(lengths),
                                      logits_mode=moin.LOGITS_ALL if last else moin.LOGITS_NONE, hidden_in=hin_gpu,
                                      hidden_out=hid, layer_begin=l, layer_end=l + 1)
        torch.cuda.synchronize()
        d = hid.double().cpu().numpy() - hin_gpu.double().cpu().numpy()
        e_blk, e_exact = rel(d, ref["hidden"] - h_in), rel(d, exact - h_in)
        e_storage = rel(ref["hidden"] - h_in, exact - h_in)   # what bf16 storage alone costs in this block
        print(f"full-width block {l}: residual update vs storage-rounded oracle {e_blk:.2e}, vs fp64 oracle "
              f"{e_exact:.2e} (storage rounding alone: {e_storage:.2e})")
        # Primary gate, against the fp64 oracle (the paper's definition, no rounding mirrored from the library):
        # the block may be no further from it than what storing its tensors in bf16 costs anyway - measured on the
        # oracle itself as the distance between its storage-rounded and exact variants - plus 10 % and 1e-3.
        assert e_exact <= 1.1 * e_storage + 1e-3, f"block {l}"
        # Secondary: distance to the storage-rounded variant.  Both sides round the same six chained tensors to
        # bf16 (norm output, q/k/v, attention output, o, gate/up product, down), but from operands that already
        # differ in their last bits, so their roundings are independent: two independent errors of size e_storage /
        # sqrt(2) each side of the common exact value give a distance of about e_storage (7.0e-3 .. 7.6e-3 here),
        # hence the bound 1.5 * 5e-3 = 7.5e-3 rather than the single-layer 5e-3.
        assert e_blk <= 1.5 * REL_FRO, f"block {l}"
        if last:
            e_log = rel(logits.double().cpu().numpy(), ref["logits"])
            print(f"full-width logits after the last block: {e_log:.2e}")
            assert e_log <= 1.5 * REL_FRO
        h_in = ref["hidden"]
    assert moin.device_status()["timeout_flag"] == 0


def test_full_forward_configuration_at_size_sampled_requests():
    """The full-forward configuration at its stated size - 22 TinyLlama-width blocks, 500 rank-64 experts on all
    seven projections (50 GB of adapter pools, 64-bit slot offsets), 64 requests x 256 tokens, all-position
    logits - against the oracle on eight sampled requests.  Experts never interact (one per request, Sec. 3.3) and
    attention is causal, so the oracle's result for the first tokens of a request, computed from host copies of
    just that request's adapters, is exact for those positions of the full batch."""
    import gc
    cfg = mi.DecoderConfig()
    R, L, N_REQ, N_TOK = 64, 256, 8, 24
    model = mi.decoder_model(cfg, seed=4, device=DEV)
    order = oracle.PROJ_ORDER
    pools = [{p: moin.Pool(model.pools[l][p].A, model.pools[l][p].B, model.pools[l][p].slot_of_expert)
              for p in order} for l in range(cfg.n_layers)]
    gm = moin.DecoderModel(cfg, model.embed, model.lm_head, model.final_norm, model.attn_norm, model.mlp_norm,
                           [{p: model.W[l][p] for p in order} for l in range(cfg.n_layers)], pools, cfg.E, cfg.scale)
    batch = mi.decoder_batch(cfg, [L] * R, seed=4, device=DEV)
    hid = torch.empty(batch.T, cfg.hidden, dtype=torch.float32, device=DEV)
    logits = moin.decoder_forward(gm, batch.tokens, batch.cu_seqlens, batch.req_expert, L, hidden_out=hid)
    torch.cuda.synchronize()
    assert moin.device_status()["timeout_flag"] == 0
    assert logits.shape == (R * L, cfg.vocab)
    # sampled requests -> host copies of their experts only
    req = np.sort(np.random.default_rng(11).choice(R, size=N_REQ, replace=False))
    re_all = batch.req_expert.cpu().numpy()
    used = sorted({int(e) for e in re_all[req] if e >= 0})
    so = model.pools[0]["q"].slot_of_expert.cpu().numpy()
    slots = torch.tensor([int(so[e]) for e in used], dtype=torch.long, device=DEV)
    so_small = np.full(cfg.E, -1, np.int32)
    so_small[used] = np.arange(len(used))
    w = {"embed": mi.bf16_bits(model.embed), "lm_head": mi.bf16_bits(model.lm_head),
         "final_norm": mi.bf16_bits(model.final_norm),
         "attn_norm": [mi.bf16_bits(t) for t in model.attn_norm], "mlp_norm": [mi.bf16_bits(t) for t in model.mlp_norm],
         "W": [{p: mi.bf16_bits(model.W[l][p]) for p in order} for l in range(cfg.n_layers)],
         "A": [{p: mi.bf16_bits(model.pools[l][p].A[slots]) for p in order} for l in range(cfg.n_layers)],
         "B": [{p: mi.bf16_bits(model.pools[l][p].B[slots]) for p in order} for l in range(cfg.n_layers)],
         "slot_of_expert": so_small}
    orc = oracle.DecoderOracle(cfg, w)
    tok_all = batch.tokens.cpu().numpy()
    rows = np.concatenate([np.arange(r * L, r * L + N_TOK) for r in req])
    sub = (tok_all[rows], np.arange(N_REQ + 1, dtype=np.int32) * N_TOK, re_all[req])
    rounded = orc.forward(*sub, round_storage=True, want_hidden=True)
    exact = orc.forward(*sub, want_hidden=True)
    ridx = torch.from_numpy(rows).long().to(DEV)
    got_l, got_h = logits[ridx].double().cpu().numpy(), hid[ridx].double().cpu().numpy()
    assert np.isfinite(got_l).all() and np.isfinite(got_h).all()
    tol = REL_FRO * np.sqrt(cfg.n_layers + 1)     # roundings of 22 blocks and the head add up like a random walk
    e_lr, e_le = rel(got_l, rounded["logits"]), rel(got_l, exact["logits"])
    e_hr, e_he = rel(got_h, rounded["hidden"]), rel(got_h, exact["hidden"])
    e_storage = rel(rounded["logits"], exact["logits"])
    print(f"full forward at size, {N_REQ} requests x first {N_TOK} tokens ({len(used)} experts): logits vs "
          f"storage-rounded oracle {e_lr:.2e}, vs fp64 oracle {e_le:.2e} (storage rounding alone {e_storage:.2e}); "
          f"hidden {e_hr:.2e} / {e_he:.2e}; gate {tol:.2e}")
    assert e_lr <= tol and e_hr <= tol
    assert e_le <= 1.1 * e_storage + tol / 2       # no further from the definition than bf16 storage explains
    # (a dropped or mis-addressed adapter would show: at s = 2 the low-rank term is 10-30 % of every projection's output)
    del gm, pools, model, logits, hid
    gc.collect()
    torch.cuda.empty_cache()
