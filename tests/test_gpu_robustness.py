"""Failure reporting, determinism and memory-safety stand-ins on the GPU, none of which faults,
traps or hangs a device: a bounded wait that runs out by design in a one-thread kernel, the same
forward twice with bit-equal results, and the guard words between workspace buffers."""
import time

import numpy as np
import pytest
import torch

from paper_2408_08146_b200 import Koala
from workloads import T7_EAGLE, TINY_EAGLE, reduced
from workloads.generate import WeightStore, prompts, random_kv, uniform_ints

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
KOALA_E_TIMEOUT = 6


def test_a_wait_that_runs_out_is_reported_through_poll():
    """The error path of the bounded waits: nothing arrives at the barrier, the wait gives up
    after a few thousand cycles, the status word takes KOALA_E_TIMEOUT and koala_poll (the same
    asynchronous copy every context uses) hands it to the host; the context stays usable."""
    cfg = TINY_EAGLE
    store = WeightStore(cfg, DEV)
    eng = Koala(cfg, store.tensors)
    assert eng.device_status() == 0
    eng.selftest_timeout(5000)
    status = 0
    for _ in range(2000):                      # poll without blocking, as a serving loop would
        done, status = eng.poll()
        if done and status != 0:
            break
        time.sleep(0.001)
    assert status == KOALA_E_TIMEOUT
    # the device and the context still work: a whole iteration runs and the code is still there
    eng.prefill(prompts(cfg), 15)
    eng.step()
    torch.cuda.synchronize()
    assert eng.device_status() == KOALA_E_TIMEOUT
    eng.close()
    # a fresh context starts clean
    eng = Koala(cfg, store.tensors)
    assert eng.device_status() == 0
    eng.close()


def _caller_tree(cfg, seed):
    N, B = cfg.N, cfg.B
    par = [-1] + [max(0, u - 1 - (u * 7) % min(u, 5)) for u in range(1, N)]
    tok = np.stack([uniform_ints(seed + b, "det.tok", N, 0, cfg.V) for b in range(B)])
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)
    return to(tok), to(np.tile(np.asarray(par), (B, 1))), to(np.full(B, N)), N


@pytest.mark.parametrize("B,N,flags", [(1, 60, 0), (2, 64, 0), (4, 64, 0), (1, 60, 4), (2, 64, 4)])
def test_same_forward_twice_is_bit_equal(B, N, flags):
    """The split-K, stream-K and 256-row-tile reductions add their partial sums in a fixed order:
    the same 7B-shaped verification (two layers; 60 rows: classic split-K and stream-K; 128 and
    256 rows: wide tiles and several token tiles) run twice gives identical bits."""
    cfg = reduced(T7_EAGLE, 2, K=1, B=B, N=N, S_max=768, prompt_len=512)
    store = WeightStore(cfg, DEV)
    eng = Koala(cfg, store.tensors, flags=flags)     # flags 4: the persistent layer kernel's stream-K sums
    eng.target_k.copy_(random_kv(cfg, "target_k", cfg.L, DEV))
    eng.target_v.copy_(random_kv(cfg, "target_v", cfg.L, DEV))
    eng.seq_len.fill_(cfg.prompt_len)
    tree = _caller_tree(cfg, 31)
    outs = []
    for _ in range(2):
        eng.koala_verify(tree)
        b = eng.buffers()
        outs.append((b["verify_logits"].clone(), b["verify_hid"].clone(), b["verify_tgt"].clone(),
                     eng.target_k[:, :, :, cfg.prompt_len:cfg.prompt_len + N].clone()))
    for a, c in zip(*outs):
        assert torch.equal(a, c)
    assert torch.isfinite(outs[0][0]).all()
    assert eng.device_status() == 0
    eng.close()


@pytest.mark.parametrize("cfg", [TINY_EAGLE, reduced(T7_EAGLE, 1, K=1, S_max=384, prompt_len=200)],
                         ids=["tiny_fp32", "t7_bf16_one_layer"])
def test_workspace_guards_stay_intact(cfg):
    """Every workspace buffer is followed by 256 guard bytes written once at init: after whole
    iterations (prompt ingestion, draft passes, expansion, verification, acceptance) none of them
    has changed, i.e. no kernel wrote past the end of its buffer."""
    store = WeightStore(cfg, DEV)
    eng = Koala(cfg, store.tensors)
    n, bad = eng.check_guards()
    assert n > 40 and bad == 0
    eng.prefill(prompts(cfg), cfg.N)
    for _ in range(2):
        eng.step()
    n2, bad = eng.check_guards()
    assert n2 == n and bad == 0
    assert eng.device_status() == 0
    eng.close()
