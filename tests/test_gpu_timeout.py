"""Failure detection on the device without a fault: every wait inside the streaming decode kernel
is bounded.  The test makes one wait run out -- the tile a CTA's consumers wait for is never
requested, and the poll limit is set to a thousand -- and checks that the kernel ends, that the
status word reports it (DYNTS_ERR_DEVICE), and that the device and the library go on working:
a fresh cache then matches the oracle."""
import numpy as np
import pytest
import torch

import workloads as W
from workloads import gen
from oracle import dynts_oracle as O
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _cfg():
    # 256 equally long slabs of 513 rows: every CTA of the streaming kernel takes one whole slab (17 chunks)
    return W.get_config("c2_llama8b").scaled(layers=32, batch=1, prompt=32, budget=512, window=32, evict_interval=64)


def _one_step_against_the_oracle(cfg, seed):
    gpu = H.make_gpu(cfg, variant=3)
    k, v = gen.torch_keys_values(cfg, seed, cfg.budget, "cuda:0")
    gpu.prefill(k, v, n_pinned=cfg.prompt)
    slabs = [(0, 0, 0), (31, 0, 7), (17, 0, 4)]
    orc = H.oracle_from_gpu(gpu, cfg, slabs=slabs)
    q, kn, vn = [x[0] for x in gen.torch_step_ring(cfg, seed, 1, "cuda:0")]
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    delta = torch.zeros((cfg.layers, cfg.batch, cfg.kv_heads, gpu.capacity), dtype=torch.float32, device="cuda:0")
    gpu.decode_attn(q, kn, vn, out, delta)
    gpu.synchronize()
    gpu.poll_error()
    G = cfg.group
    qh, kh, vh = q.double().cpu().numpy(), kn.double().cpu().numpy(), vn.double().cpu().numpy()
    og, dh = out.float().cpu().numpy(), delta.cpu().numpy()
    for (l, b, h) in slabs:
        sl = orc.slab(l, b, h)
        sl.K[sl.n], sl.V[sl.n] = kh[l, b, h], vh[l, b, h]
        n = sl.n + 1
        alpha = O.attention_weights(qh[l, b, h * G:(h + 1) * G], sl.K[:n])
        assert H.rel_err_vectors(og[l, b, h * G:(h + 1) * G], O.attention_output(alpha, sl.V[:n])) <= H.TOL_OUT["bf16"]
        assert float(np.abs(dh[l, b, h, :n] - alpha.sum(axis=0)).max()) <= H.TOL_DELTA
    gpu.close()


@pytest.mark.parametrize("item", [0, 5])
def test_a_wait_that_runs_out_is_reported_and_nothing_hangs(item):
    import paper_2601_18383_b200 as D
    cfg = _cfg()
    gpu = H.make_gpu(cfg, variant=3)
    k, v = gen.torch_keys_values(cfg, 9100, cfg.budget, "cuda:0")
    gpu.prefill(k, v, n_pinned=cfg.prompt)
    q, kn, vn = [x[0] for x in gen.torch_step_ring(cfg, 9100, 1, "cuda:0")]
    out = torch.empty((cfg.layers, cfg.batch, cfg.q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda:0")
    gpu.decode_attn(q, kn, vn, out)                      # an ordinary step first
    gpu.synchronize()
    gpu.poll_error()
    with pytest.raises(D.DyntsError):
        gpu.set_wait_limit(3)                            # below the smallest limit the library accepts
    gpu.set_wait_limit(1000)
    gpu.debug_drop_tile_load(item)                       # one-shot: the next launch's first CTA never asks for that tile
    gpu.decode_attn(q, kn, vn, out)
    torch.cuda.synchronize()                             # the kernel ended by itself
    with pytest.raises(D.DyntsError) as e:
        gpu.poll_error()
    assert e.value.status == D.DYNTS_ERR_DEVICE
    word = int(str(e.value).split("status word 0x")[1].split()[0], 16)
    assert word & 8                                      # the timeout bit
    gpu.close()
    # the context is intact: a fresh cache computes a correct step
    _one_step_against_the_oracle(cfg, 9101)


def test_the_default_limit_is_never_reached_by_an_ordinary_run():
    cfg = _cfg()
    _one_step_against_the_oracle(cfg, 9102)
