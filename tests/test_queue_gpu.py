"""GPU tests of the bounded request queue in front of a real handle: requests pushed by several
threads, in any grouping and in both serving modes, deliver exactly the bits the handle delivers
for each environment alone (paper sections 4.2.2 and 4.2.3)."""
import threading

import numpy as np
import pytest
import torch

from paper_2609_27547_b200 import binding as B
from paper_2609_27547_b200 import synth
from gpu_helpers import Runner, TOL, stack
from helpers import chunk_rel_err, oracle_run

pytestmark = pytest.mark.gpu
SEED = 777


@pytest.mark.parametrize("dtype,step_mode", [("f32", False), ("f32", True), ("bf16", False), ("bf16", True)])
def test_queue_serves_the_same_bits_as_direct_submits(dtype, step_mode):
    w = synth.scaled(synth.WORKLOADS[0], B=24, dtype=dtype, P=(10, 120), mixed_steps=True)
    wt = synth.make_weights(w, SEED, random_gains=True)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    ids = list(range(w.B))
    r = Runner(w, wt, envs, max_inflight_groups=1, max_group_envs=8)
    direct = stack(r.run([ids[i:i + 8] for i in range(0, w.B, 8)], quota=74), ids)
    assert chunk_rel_err(direct, oracle_run(w, wt, envs)) <= TOL[dtype]
    stream = torch.cuda.Stream()
    q = B.Queue(r.gen, capacity=6, max_group=8, sm_quota=74, step_mode=step_mode, linger_us=200, stream=stream)
    outs = {e: torch.empty_like(r.noise[e]) for e in ids}
    tickets = {}

    def simulator(mine):
        for e in mine:
            tickets[e] = q.push(e, r.kv[e], envs[e].P, r.noise[e], outs[e], envs[e].step)

    threads = [threading.Thread(target=simulator, args=(ids[i::4],)) for i in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    for e in ids:
        assert q.wait(tickets[e]) == B.OK
    st = q.stats()
    q.destroy()
    got = np.stack([outs[e].cpu().numpy() for e in ids])
    assert np.array_equal(got, direct)
    assert st["completed"] == w.B and st["failed"] == 0 and st["max_waiting"] <= 6
    if step_mode:
        assert st["group_envs"] == sum(w.K - e.step for e in envs)       # one submit row per remaining Euler step
    else:
        assert st["group_envs"] == w.B
    r.close()


def test_scattered_submit_checks_its_pointers():
    w = synth.scaled(synth.WORKLOADS[0], B=2)
    wt = synth.make_weights(w, SEED)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    r = Runner(w, wt, envs)
    import ctypes as C
    L = B.lib()
    ids = (C.c_int64 * 2)(0, 1)
    kv = (C.c_void_p * 2)(r.kv[0].data_ptr(), r.kv[1].data_ptr())
    out = torch.empty(2, w.H, w.A, device="cuda")
    good = (C.c_void_p * 2)(r.noise[0].data_ptr(), r.noise[1].data_ptr())
    outp = (C.c_void_p * 2)(out[0].data_ptr(), out[1].data_ptr())
    bad = (C.c_void_p * 2)(r.noise[0].data_ptr(), None)
    odd = (C.c_void_p * 2)(r.noise[0].data_ptr(), r.noise[1].data_ptr() + 2)
    assert L.ebrl_actgen_submit_scattered(r.gen._h, 2, ids, kv, bad, outp, 0, None, None) == B.ERR_INVALID_ARG
    assert L.ebrl_actgen_submit_scattered(r.gen._h, 2, ids, kv, odd, outp, 0, None, None) == B.ERR_INVALID_ARG
    assert L.ebrl_actgen_submit_scattered(r.gen._h, 2, ids, kv, None, outp, 0, None, None) == B.ERR_INVALID_ARG
    assert L.ebrl_actgen_submit_scattered(r.gen._h, 0, ids, kv, None, None, 0, None, None) == B.OK
    assert L.ebrl_actgen_submit_scattered(r.gen._h, 2, ids, kv, good, outp, 0, None, None) == B.OK
    r.gen.sync()
    ref = stack(r.run([[0, 1]]), [0, 1])
    assert np.array_equal(out.cpu().numpy(), ref)
    assert L.ebrl_actgen_k_steps(r.gen._h) == w.K and L.ebrl_actgen_k_steps(None) == 0
    r.close()
