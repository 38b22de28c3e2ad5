"""GPU parity of the Importance Predictor head (Section 4.1, Eq. 7; Appendix A: d -> 2d -> d/2 -> 1)
against the float64 oracle on bf16-representable weights and hidden states."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import dynts_oracle as O

pytestmark = pytest.mark.gpu


def _params(d, batch, seed):
    r = np.random.default_rng(seed)
    bf = lambda x: W.to_cache_dtype(x, "bf16")
    h = bf(r.standard_normal((batch, d)))
    W1 = bf(r.standard_normal((2 * d, d)) / np.sqrt(d))
    W2 = bf(r.standard_normal((d // 2, 2 * d)) / np.sqrt(2 * d))
    W3 = bf(r.standard_normal((1, d // 2)) / np.sqrt(d // 2))
    b1 = r.standard_normal(2 * d).astype(np.float32) * 0.1
    b2 = r.standard_normal(d // 2).astype(np.float32) * 0.1
    b3 = r.standard_normal(1).astype(np.float32)
    return h, W1, b1, W2, b2, W3, b3


@pytest.mark.parametrize("d,batch,act", [(512, 1, "none"), (512, 3, "relu"), (1024, 8, "relu"), (1536, 11, "none"),
                                         (3584, 4, "relu"), (4096, 8, "relu"), (4096, 17, "none")])
def test_predictor_mlp_matches_oracle(d, batch, act):
    import paper_2601_18383_b200 as D
    h, W1, b1, W2, b2, W3, b3 = _params(d, batch, 100 + d + batch)
    ref = O.predictor_mlp(h, W1, b1, W2, b2, W3, b3, act)
    dev16 = lambda x: torch.from_numpy(x).to(torch.bfloat16).cuda().contiguous()
    dev32 = lambda x: torch.from_numpy(x).cuda().contiguous()
    nbytes = D.dynts_predictor_mlp_scratch_bytes(d, batch)
    assert nbytes > 0
    scratch = torch.full((nbytes // 4,), float("nan"), dtype=torch.float32, device="cuda:0")   # contents must not matter
    scores = torch.zeros(batch, dtype=torch.float32, device="cuda:0")
    args = (dev16(h), dev16(W1), dev32(b1), dev16(W2), dev32(b2), dev16(W3), dev32(b3))
    for _ in range(2):
        D.dynts_predictor_mlp(*args, d, batch, 1 if act == "relu" else 0, scratch, nbytes, scores,
                              torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    got = scores.cpu().numpy().astype(np.float64)
    # fp32 accumulation of up to 8192 products of O(1/sqrt(K)) terms: a few 1e-6 in practice
    assert np.abs(got - ref).max() <= 1e-4 * max(1.0, np.abs(ref).max()), (got, ref)
    # biases are optional
    D.dynts_predictor_mlp(args[0], args[1], None, args[3], None, args[5], None, d, batch, 1 if act == "relu" else 0,
                          scratch, nbytes, scores, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    z = lambda x: np.zeros_like(x)
    ref0 = O.predictor_mlp(h, W1, z(b1), W2, z(b2), W3, z(b3), act)
    assert np.abs(scores.cpu().numpy() - ref0).max() <= 1e-4 * max(1.0, np.abs(ref0).max())


def test_predictor_argument_checks_and_scores_feed_the_cache():
    import paper_2601_18383_b200 as D
    from tests import helpers as H
    assert D.dynts_predictor_mlp_scratch_bytes(500, 2) == 0
    d, batch = 512, 2
    h, W1, b1, W2, b2, W3, b3 = _params(d, batch, 7)
    dev16 = lambda x: torch.from_numpy(x).to(torch.bfloat16).cuda().contiguous()
    nbytes = D.dynts_predictor_mlp_scratch_bytes(d, batch)
    scratch = torch.empty(nbytes, dtype=torch.uint8, device="cuda:0")
    scores = torch.zeros(batch, dtype=torch.float32, device="cuda:0")
    with pytest.raises(D.DyntsError):
        D.dynts_predictor_mlp(dev16(h), dev16(W1), None, dev16(W2), None, dev16(W3), None, d, batch, 0, scratch, nbytes - 16,
                              scores, None)
    with pytest.raises(D.DyntsError):
        D.dynts_predictor_mlp(dev16(h), dev16(W1), None, dev16(W2), None, dev16(W3), None, d, batch, 5, scratch, nbytes, scores, None)
    cfg = W.get_config("c2_llama8b").scaled(layers=1, batch=batch, prompt=16, budget=64, window=8, evict_interval=4)
    gpu = H.make_gpu(cfg)
    gpu.set_score_source(D.DYNTS_SCORE_EXTERNAL)
    pk, pv = W.prompt_kv(cfg, 1)
    gpu.prefill(H.dev(pk, cfg), H.dev(pv, cfg))
    q, k, v = [H.dev(x, cfg) for x in W.DecodeStream(cfg, 1).step(1)]
    out = torch.empty((1, batch, cfg.q_heads, 128), dtype=torch.bfloat16, device="cuda:0")
    gpu.decode_attn(q, k, v, out)
    st = torch.cuda.current_stream().cuda_stream
    D.dynts_predictor_mlp(dev16(h), dev16(W1), None, dev16(W2), None, dev16(W3), None, d, batch, 0, scratch, nbytes, scores, st)
    gpu.append_scores(scores)
    gpu.synchronize()
    ref = O.predictor_mlp(h, W1, np.zeros(2 * d), W2, np.zeros(d // 2), W3, np.zeros(1), "none")
    got = gpu.scores_tensor()[0, :, :, 16].cpu().numpy()
    assert np.abs(got - ref[:, None]).max() <= 1e-4
    gpu.close()
