"""The DLLM_TIMEOUT path of the bounded device-side waits, exercised without faulting or hanging anything:
a host-set flag makes the first CTA of a GEMM launch leave out one tile copy, so one pipeline stage never
completes and that CTA's waits run into a limit shortened to a few milliseconds.  The CTA must record the
status, skip its epilogue, free its tensor memory and return; the host must read DLLM_TIMEOUT once, and the
next call on the same stream, session and context must work as if nothing had happened.  Collected near the
end so that it runs after the parity tests proper."""
import numpy as np
import pytest

from oracle import dllm_oracle as O
from paper_2506_06295_b200 import synth
from tests.helpers import rel_l2

pytestmark = pytest.mark.gpu
LIMIT_NS = 3_000_000      # 3 ms per wait


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2506_06295_b200 import build as build_mod
    build_mod.build()
    from paper_2506_06295_b200 import dllm
    assert torch.cuda.is_available()
    yield torch, dllm
    dllm.debug_skip_one_load(False)          # whatever a failing test left behind
    dllm.debug_set_wait_limit_ns(0)


def test_kernel_level_wait_runs_out_and_the_next_call_is_clean(env):
    torch, dllm = env
    A = torch.from_numpy(synth.round_to_bf16(synth.random_normal((40, 256), seed=5))).cuda().to(torch.bfloat16)
    W = torch.from_numpy(synth.round_to_bf16(synth.random_normal((384, 256), seed=6))).cuda().to(torch.bfloat16)
    want = A.double().cpu().numpy() @ W.double().cpu().numpy().T
    dllm.kernel_status()                      # clean to start with
    dllm.debug_set_wait_limit_ns(LIMIT_NS)
    dllm.debug_skip_one_load(True)
    try:
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        dllm.gemm_bf16(A, W)                  # returns normally: the call only enqueues
        t1.record()
        with pytest.raises(dllm.DllmError) as e:
            dllm.kernel_status()
        assert e.value.status == dllm.TIMEOUT
        assert 0.5 * LIMIT_NS / 1e6 < t0.elapsed_time(t1) < 1000.0      # the wait ended at its limit, not at 2 s
    finally:
        dllm.debug_skip_one_load(False)
        dllm.debug_set_wait_limit_ns(0)
    dllm.kernel_status()                      # the word was cleared by the read
    got = dllm.gemm_bf16(A, W).cpu().numpy()
    dllm.kernel_status()
    assert rel_l2(got, want) < 1e-5


def test_session_reports_timeout_once_and_then_steps_normally(env):
    torch, dllm = env
    cfg = synth.small_bf16_model()
    B, P, R = 1, 96, 40
    w = synth.make_weights(cfg)
    prompt = synth.make_prompt(cfg, B, P)
    orc = O.DLLMOracle(cfg, w, B, P, R, dtype=np.float32)
    orc.set_prompt(prompt)
    r = orc.step(True, True)
    ses = dllm.Session(dllm.Model(cfg).load(w), B, P, R)
    ses.set_prompt(prompt)
    dllm.debug_set_wait_limit_ns(LIMIT_NS)
    dllm.debug_skip_one_load(True)
    try:
        ses.step_full()                        # every projection's first CTA gives up after the limit
        with pytest.raises(dllm.DllmError) as e:
            ses.sync()
        assert e.value.status == dllm.TIMEOUT and "wait" in str(e.value)
    finally:
        dllm.debug_skip_one_load(False)
        dllm.debug_set_wait_limit_ns(0)
    ses.sync()                                 # read once, cleared
    ses.set_prompt(prompt)
    ses.step_full()
    ses.sync()
    assert rel_l2(ses.hidden(), r.hidden) < 2e-2
