"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle element by
element on the same seeded inputs; bit-identity of GPU results across SM quotas, group
partitions, arrival orders and step-at-a-time batching; closed forms; edge cases.

Tolerances (max over environments of max|gpu - oracle| / max(1, max|oracle|) on the final
action chunk): 1e-4 for fp32 models, 2e-2 for bf16 models with fp32 accumulation.
"""
import numpy as np
import pytest
import torch

from paper_2609_27547_b200 import binding as B
from paper_2609_27547_b200 import synth
from helpers import chunk_rel_err, oracle_run, np32
from gpu_helpers import Runner, TOL, stack, to_dev

pytestmark = pytest.mark.gpu
SEED = synth.DEFAULT_SEED


def _setup(w, n=None, random_gains=True, seed=SEED):
    wt = synth.make_weights(w, seed, random_gains=random_gains)
    envs = [synth.make_env(w, e, seed) for e in range(n if n is not None else w.B)]
    return wt, envs


def test_cfg0_tiny_fp32_parity():
    """The tiny fp32 configuration as stated: 16 envs, one group, full quota."""
    w = synth.WORKLOADS[0]
    wt, envs = _setup(w, random_gains=False)
    ref = oracle_run(w, wt, envs)
    r = Runner(w, wt, envs)
    got = stack(r.run([list(range(w.B))]), range(w.B))
    r.close()
    assert chunk_rel_err(got, ref) <= TOL["f32"]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_small_models_parity_ragged(dtype):
    """Several row tiles and a ragged tail: 37 envs x H=8 = 296 rows (128-row tiles: 2 full +
    40 rows), ragged prefix lengths not multiples of the key block, mixed step indices."""
    w = synth.scaled(synth.WORKLOADS[0], B=37, dtype=dtype, P=(1, 97), mixed_steps=True, K=5)
    wt, envs = _setup(w)
    ref = oracle_run(w, wt, envs)
    r = Runner(w, wt, envs)
    got = stack(r.run([list(range(w.B))]), range(w.B))
    r.close()
    assert chunk_rel_err(got, ref) <= TOL[dtype]


def test_every_gemm_tile_shape_every_row_against_the_oracle(monkeypatch):
    """The three tensor-core GEMM tile shapes forced in turn (CTA pairs on 256 x 256 tiles, one CTA on
    128 x 256, one CTA on 128 x 128) on a batch of 43 envs x H=16 = 688 rows: two full 256-row pair
    tiles plus a tail whose leader CTA is full and whose peer CTA holds 48 rows, and 128-row tiles 5 full
    + 48.  EVERY row is compared with the oracle, and the three shapes with each other bit for bit
    (each output element accumulates over k in the same order whatever the tile)."""
    w = synth.scaled(synth.WORKLOADS[0], B=43, dtype="bf16", H=16, A=14, d=512, n_heads=8, L=2, K=3, P=(5, 90),
                     mixed_steps=True)
    wt, envs = _setup(w)
    ref = oracle_run(w, wt, envs)
    ids = list(range(w.B))
    got = {}
    for shape in ("2", "256", "128"):
        monkeypatch.setenv("EBRL_GEMM_SHAPE", shape)    # read when the handle is created
        r = Runner(w, wt, envs)
        got[shape] = stack(r.run([ids]), ids)
        if shape == "2":
            assert np.array_equal(stack(r.run([ids], quota=37), ids), got[shape])   # 18 pairs instead of 74
        r.close()
        assert chunk_rel_err(got[shape], ref) <= TOL["bf16"], "tile shape %s" % shape
    monkeypatch.delenv("EBRL_GEMM_SHAPE")
    assert np.array_equal(got["2"], got["256"]) and np.array_equal(got["2"], got["128"])
    r = Runner(w, wt, envs)                              # and the shapes the library picks by itself
    assert np.array_equal(stack(r.run([ids]), ids), got["2"])
    r.close()


def test_fp32_projections_on_tensor_cores_and_on_the_plain_alus():
    """fp32 models run their projections on the tensor cores (every operand the exact sum of three
    bf16 terms, six products per term pair) unless told to use the FFMA kernels.  Both must stay
    within the fp32 bound of the oracle on a model with long reductions (d = 512, MLP width 2048),
    several row tiles and a ragged tail; the tensor-core path must also be quota-independent."""
    w = synth.scaled(synth.WORKLOADS[0], B=37, dtype="f32", d=512, n_heads=8, L=3, K=4, P=(1, 97), mixed_steps=True)
    wt, envs = _setup(w)
    ref = oracle_run(w, wt, envs)
    ids = list(range(w.B))
    r = Runner(w, wt, envs)
    got = stack(r.run([ids]), ids)
    assert chunk_rel_err(got, ref) <= TOL["f32"]
    for q in (16, 37, 74):
        assert np.array_equal(stack(r.run([ids], quota=q), ids), got)
    assert np.array_equal(stack(r.run([ids[:9], ids[9:]]), ids), got)
    r.close()
    r = Runner(w, wt, envs, flags=B.FLAG_FORCE_SIMT)
    alu = stack(r.run([ids]), ids)
    r.close()
    assert chunk_rel_err(alu, ref) <= TOL["f32"]
    print("fp32 max chunk-relative error: tensor cores %.2e, FFMA %.2e" % (chunk_rel_err(got, ref), chunk_rel_err(alu, ref)))


@pytest.mark.parametrize("H,A,P", [(8, 7, (15, 17)), (5, 3, (1, 40)), (1, 2, (1, 3)), (8, 7, (250, 530)), (7, 7, (16, 16))])
def test_fp32_warp_per_item_attention_edge_shapes(H, A, P):
    """The fp32 attention kernel that gives every (environment, head) to one warp (head_dim 64, H <= 8):
    fewer than eight query rows, prefixes shorter than / equal to / just past one 16-key stage and many
    stages long, more items than warps so that a warp's copies run on into its next item (whose prefix
    length differs).  Against the oracle, across quotas, and alone."""
    w = synth.scaled(synth.WORKLOADS[0], B=41, dtype="f32", H=H, A=A, P=P, K=3, mixed_steps=True)
    wt, envs = _setup(w)
    ref = oracle_run(w, wt, envs)
    ids = list(range(w.B))
    r = Runner(w, wt, envs)
    got = stack(r.run([ids]), ids)
    assert chunk_rel_err(got, ref) <= TOL["f32"]
    for q in (2, 5, 148):                 # 2 CTAs x 8 warps for 164 items: about ten items per warp
        assert np.array_equal(stack(r.run([ids], quota=q), ids), got), "quota %d" % q
    assert np.array_equal(stack(r.run([[e] for e in ids[:5]] + [ids[5:]], quota=3), ids), got)
    r.close()
    r = Runner(w, wt, envs, flags=B.FLAG_FORCE_SIMT)   # the block-per-four-items kernel on the same inputs
    alu = stack(r.run([ids]), ids)
    r.close()
    assert chunk_rel_err(alu, ref) <= TOL["f32"]


def test_fp32_other_head_dims_take_the_general_attention_kernel():
    """head_dim 32 and 128 in fp32 are outside the warp-per-item kernel: the general one serves them."""
    for d, nh in ((128, 4), (256, 2)):
        w = synth.scaled(synth.WORKLOADS[0], B=11, dtype="f32", d=d, n_heads=nh, P=(3, 70), mixed_steps=True)
        wt, envs = _setup(w)
        ref = oracle_run(w, wt, envs)
        r = Runner(w, wt, envs)
        got = stack(r.run([list(range(w.B))]), range(w.B))
        r.close()
        assert chunk_rel_err(got, ref) <= TOL["f32"]


def test_fp32_tensor_core_gemm_on_pairs_and_on_single_ctas_agree(monkeypatch):
    """The fp32 tensor-core GEMM runs on CTA pairs (256 x 256 tiles) or on single CTAs (128 x 128), chosen per
    projection; forced in turn (`EBRL_GEMM_SHAPE` = 2 / 128, read when the handle is created) on 37 envs x H = 8
    = 296 rows (one full 256-row pair tile plus a 40-row tail in the leader CTA only) of a d = 512 model: each
    against the oracle, and bit-identical to each other and to the library's own choice at several quotas."""
    w = synth.scaled(synth.WORKLOADS[0], B=37, dtype="f32", d=512, n_heads=8, L=2, K=3, P=(1, 97), mixed_steps=True)
    wt, envs = _setup(w)
    ref = oracle_run(w, wt, envs)
    ids = list(range(w.B))
    got = {}
    for shape in ("128", "2"):
        monkeypatch.setenv("EBRL_GEMM_SHAPE", shape)
        r = Runner(w, wt, envs)
        got[shape] = stack(r.run([ids]), ids)
        assert np.array_equal(stack(r.run([ids], quota=5), ids), got[shape])
        r.close()
        assert chunk_rel_err(got[shape], ref) <= TOL["f32"], shape
    assert np.array_equal(got["128"], got["2"])
    monkeypatch.delenv("EBRL_GEMM_SHAPE")
    r = Runner(w, wt, envs)
    for q in (0, 2, 3, 16):
        assert np.array_equal(stack(r.run([ids], quota=q), ids), got["2"]), "quota %d" % q
    r.close()


def test_bf16_plain_alu_kernels_parity():
    """The bf16 model on the plain-ALU kernels (the path taken when d is not a multiple of 256,
    and on request)."""
    w = synth.scaled(synth.WORKLOADS[0], B=19, dtype="bf16", d=128, n_heads=4, P=(3, 70), mixed_steps=True)
    wt, envs = _setup(w)
    ref = oracle_run(w, wt, envs)
    r = Runner(w, wt, envs)
    got = stack(r.run([list(range(w.B))]), range(w.B))
    r.close()
    assert chunk_rel_err(got, ref) <= TOL["bf16"]
    w = synth.scaled(w, d=256)
    wt, envs = _setup(w)
    r = Runner(w, wt, envs, flags=B.FLAG_FORCE_SIMT)
    got = stack(r.run([list(range(w.B))]), range(w.B))
    r.close()
    assert chunk_rel_err(got, oracle_run(w, wt, envs)) <= TOL["bf16"]


def test_cfg1_model_bf16_parity_sample():
    """The mid-size bf16 head (d=1024, L=4, 16 heads, P=256, K=10) on a few environments."""
    w = synth.scaled(synth.WORKLOADS[1], B=6)
    wt = synth.make_weights(w, SEED, device="cuda")
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    ref = oracle_run(w, wt, envs)
    r = Runner(w, wt, envs)
    got = stack(r.run([list(range(w.B))]), range(w.B))
    r.close()
    assert chunk_rel_err(got, ref) <= TOL["bf16"]


def test_bimanual_shape_bf16_parity():
    """H=16, A=14, head_dim=128 (the large configuration's token and head shapes) at d=256."""
    w = synth.scaled(synth.WORKLOADS[4], B=9, d=256, n_heads=2, L=2, P=(40, 70), K=3, group=None)
    wt, envs = _setup(w)
    ref = oracle_run(w, wt, envs)
    r = Runner(w, wt, envs)
    got = stack(r.run([list(range(w.B))]), range(w.B))
    r.close()
    assert chunk_rel_err(got, ref) <= TOL["bf16"]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_bit_identity_across_quotas_partitions_orders(dtype):
    """Same environments: one group, seeded ragged groups, a second grouping, reversed order,
    each alone, and SM quotas 16/37/74/148 must give the same bits."""
    w = synth.scaled(synth.WORKLOADS[2], B=40, dtype=dtype, P=(64, 160), group=(1, 12))
    wt, envs = _setup(w)
    ids = list(range(w.B))
    r = Runner(w, wt, envs, max_inflight_groups=3)
    base = stack(r.run([ids], quota=0), ids)
    for q in (16, 37, 74, 148):
        assert np.array_equal(stack(r.run([ids], quota=q), ids), base), "quota %d" % q
    g1 = synth.arrival_groups(w, SEED)
    g2 = synth.arrival_groups(w, SEED + 1)
    assert len(g1) > 3 and g1 != g2
    assert np.array_equal(stack(r.run(g1, quota=37), ids), base)
    assert np.array_equal(stack(r.run(g2, quota=74), ids), base)
    assert np.array_equal(stack(r.run([ids[::-1]]), ids), base)
    assert np.array_equal(stack(r.run([[e] for e in ids[:10]], quota=16), ids[:10]), base[:10])
    # and against the oracle
    assert chunk_rel_err(base, oracle_run(w, wt, envs)) <= TOL[dtype]
    r.close()


def test_step_at_a_time_equals_full_run():
    """n_steps = 1 re-batching every Euler step (state carried by the caller in fp32) gives the
    same bits as running each environment to the end in one submit."""
    w = synth.scaled(synth.WORKLOADS[0], B=12, P=(20, 50), mixed_steps=True, K=4)
    wt, envs = _setup(w)
    ids = list(range(w.B))
    r = Runner(w, wt, envs)
    full = stack(r.run([ids]), ids)
    state = {e: r.noise[e].clone() for e in ids}
    steps = {e: r.envs[e].step for e in ids}
    live = list(ids)
    while live:
        res = r.run([live], n_steps=1, state=state, steps=steps)
        for e in live:
            state[e] = torch.from_numpy(res[e]).cuda()
            steps[e] += 1
        live = [e for e in live if steps[e] < w.K]
    assert np.array_equal(np.stack([state[e].cpu().numpy() for e in ids]), full)
    r.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_zero_weights_closed_form(dtype):
    """All matrices zero: a_K = a_0 + b (K additions of b/K in fp32)."""
    w = synth.scaled(synth.WORKLOADS[0], B=5, dtype=dtype)
    wt, envs = _setup(w)
    for k in ("w_in", "w_out"):
        wt[k].zero_()
    for l in wt["layers"]:
        for k in ("w_qkv", "w_o", "w_qc", "w_oc", "w_1", "w_2"):
            l[k].zero_()
    r = Runner(w, wt, envs)
    got = stack(r.run([list(range(w.B))]), range(w.B))
    r.close()
    want = np.stack([np32(e.noise) for e in envs]).astype(np.float64) + np32(wt["b_out"]).astype(np.float64)
    assert np.abs(got - want).max() < 1e-6


def test_pull_field_closed_form():
    """v = c - a: a_K = c + (a_0 - c)(1 - 1/K)^K; from step k0 the exponent is K - k0."""
    w = synth.scaled(synth.WORKLOADS[0], B=7, K=10, mixed_steps=True)
    wt, envs = _setup(w)
    r = Runner(w, wt, envs, flags=B.FLAG_TEST_PULL)
    got = stack(r.run([list(range(w.B))]), range(w.B))
    r.close()
    c = np32(wt["b_out"]).astype(np.float64)
    for i, e in enumerate(envs):
        want = c + (np32(e.noise).astype(np.float64) - c) * (1 - 1 / w.K) ** (w.K - e.step)
        assert np.abs(got[i] - want).max() < 1e-6


def test_edge_cases():
    """Empty group; one environment; prefix of one token; H = 1; one Euler step."""
    w = synth.scaled(synth.WORKLOADS[0], B=3, H=1, A=1, P=(1, 1), K=1)
    wt, envs = _setup(w)
    r = Runner(w, wt, envs)
    assert r.run([[]]) == {}
    got = stack(r.run([[0], [1, 2]]), range(3))
    r.close()
    assert chunk_rel_err(got, oracle_run(w, wt, envs)) <= TOL["f32"]


def test_maximum_sizes_of_the_interface():
    """H = 32 and A = 32 (the largest supported), head_dim 32, prefix longer than several key
    blocks."""
    w = synth.scaled(synth.WORKLOADS[0], B=3, H=32, A=32, d=128, n_heads=4, L=1, P=(130, 200), K=2)
    wt, envs = _setup(w)
    r = Runner(w, wt, envs)
    got = stack(r.run([[0, 1, 2]]), range(3))
    r.close()
    assert chunk_rel_err(got, oracle_run(w, wt, envs)) <= TOL["f32"]


def test_host_buffer_entry_point_matches_device_entry_point():
    w = synth.scaled(synth.WORKLOADS[0], B=6, P=(10, 40), mixed_steps=True)
    wt, envs = _setup(w)
    ids = list(range(w.B))
    r = Runner(w, wt, envs)
    base = stack(r.run([ids]), ids)
    noise = torch.stack([e.noise for e in envs]).pin_memory()
    out = torch.empty_like(noise).pin_memory()
    kv = [e.kv.contiguous().pin_memory() for e in envs]
    r.gen.submit_host(ids, kv, noise, out, step_index=[e.step for e in envs])
    r.gen.sync()
    assert np.array_equal(out.numpy(), base)
    r.close()


def test_errors_and_busy_ids():
    w = synth.scaled(synth.WORKLOADS[0], B=4)
    wt, envs = _setup(w)
    r = Runner(w, wt, envs, max_inflight_groups=2)
    noise = torch.stack([r.noise[e] for e in range(4)])
    out = torch.empty_like(noise)
    kv = [r.kv[e] for e in range(4)]
    with pytest.raises(B.EbrlError) as ei:
        r.gen.submit([0, 1, 1, 2], kv, noise, out)
    assert ei.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.EbrlError) as ei:
        r.gen.submit([0, 1, 2, 3], kv, noise, out, sm_quota=100000)
    assert ei.value.status == B.ERR_QUOTA
    with pytest.raises(B.EbrlError) as ei:
        r.gen.submit([0, 1, 2, 3], kv, noise, out, step_index=[0, 0, w.K, 0])
    assert ei.value.status == B.ERR_INVALID_ARG
    r.gen.submit([0, 1, 2, 3], kv, noise, out)
    out2 = torch.empty_like(noise)
    with pytest.raises(B.EbrlError) as ei:
        r.gen.submit([7, 3], kv[:2], noise[:2], out2[:2])      # env 3 is still in flight
    assert ei.value.status == B.ERR_ENV_BUSY
    r.gen.sync()
    r.gen.submit([7, 3], kv[:2], noise[:2].contiguous(), out2[:2])   # fine after the sync
    r.gen.sync()
    st = r.gen.stats()
    assert st["groups"] == 2 and st["envs"] == 6 and st["kernel_launches"] > 0
    r.close()


def test_bounded_wait_times_out_cleanly_and_context_survives():
    """A wait that nothing satisfies gives up after its limit with EBRL_ERR_TIMEOUT in the status
    word -- no trap, no hang -- and the device keeps working afterwards."""
    rc, st, waited = B.wait_probe(50_000_000, signal_it=True)
    assert rc == B.OK and st == B.OK and waited < 10_000_000
    rc, st, waited = B.wait_probe(50_000_000, signal_it=False)          # 50 ms limit, nobody arrives
    assert rc == B.OK and st == B.ERR_TIMEOUT
    assert 40_000_000 <= waited <= 500_000_000
    # the context is still usable: run a normal group
    w = synth.scaled(synth.WORKLOADS[0], B=3)
    wt, envs = _setup(w)
    r = Runner(w, wt, envs)
    got = stack(r.run([[0, 1, 2]]), range(3))
    r.close()
    assert chunk_rel_err(got, oracle_run(w, wt, envs)) <= TOL["f32"]
    rc, _, _ = B.wait_probe(0, False)
    assert rc == B.ERR_INVALID_ARG


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_sm_partition_gives_the_same_bits(dtype):
    """With EBRL_FLAG_GREEN_CTX every batch runs inside a driver-enforced SM partition of at least
    sm_quota SMs (where the driver offers green contexts; otherwise the grid cap alone applies).
    Either way the results are the bits of the unpartitioned run."""
    w = synth.scaled(synth.WORKLOADS[2], B=24, dtype=dtype, P=(64, 130), group=(1, 9))
    wt, envs = _setup(w)
    ids = list(range(w.B))
    r = Runner(w, wt, envs)
    base = stack(r.run([ids]), ids)
    r.close()
    r = Runner(w, wt, envs, flags=B.FLAG_GREEN_CTX, max_inflight_groups=2)
    for q in (16, 37, 74):
        got = stack(r.run(synth.arrival_groups(w, SEED), quota=q), ids)
        assert np.array_equal(got, base), "quota %d" % q
        st = r.gen.stats()
        assert st["granted_sms"] == q
        if st["green_ctx_active"]:
            assert q <= st["green_ctx_sms"] <= 148
            # the complementary partition: the other SMs, with a stream a co-runner can be fenced into
            gen_sms, rest_sms, rest_stream = r.gen.partition_info(q)
            assert gen_sms == st["green_ctx_sms"] and gen_sms + rest_sms == 148 and rest_stream
            buf = torch.zeros(1 << 20, device="cuda")
            B.sim_corunner_launch(buf, 2, rest_sms, r.gen.rest_stream(q))      # runs there beside nothing: just must work
            r.gen.rest_stream(q).synchronize()
            assert torch.allclose(buf, torch.full_like(buf, 0.001 * 0.999 + 0.001))
    assert r.gen.partition_info(148) == (0, 0, None)  # the whole chip needs no partition
    got = stack(r.run([ids], quota=0), ids)          # full chip: no partition needed
    assert np.array_equal(got, base) and r.gen.stats()["green_ctx_active"] == 0
    r.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_per_layer_prefix_planes(dtype):
    """kv_layers = n_layers: every layer cross-attends to its own K/V plane pair
    ([L][2][P][d] per environment) instead of one shared pair."""
    import oracle
    from helpers import oracle_cfg, oracle_weights
    w = synth.scaled(synth.WORKLOADS[0], B=7, dtype=dtype, L=3, P=(9, 70), mixed_steps=True)
    wt = synth.make_weights(w, SEED, random_gains=True)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    kvs = [synth.normal(SEED, "kv_per_layer", e.env_id, (w.L, 2, e.P, w.d), dtype=w.torch_dtype) for e in envs]
    oc = oracle_cfg(w)
    oc.kv_layers = w.L
    ref = oracle.actgen(oc, oracle_weights(wt), [np32(k) for k in kvs], np.stack([np32(e.noise) for e in envs]),
                        step_index=[e.step for e in envs])
    cfg = B.cfg_for(w, max_group_envs=w.B, max_inflight_groups=2)
    cfg.kv_layers = w.L
    cfg.max_prefix_len = 70
    gen = B.ActGen(cfg, wt)
    noise = torch.stack([e.noise for e in envs]).cuda()
    out = torch.empty_like(noise)
    dkv = [k.cuda() for k in kvs]
    gen.submit(list(range(4)), dkv[:4], noise[:4], out[:4], sm_quota=37, step_index=[e.step for e in envs[:4]])
    gen.submit(list(range(4, 7)), dkv[4:], noise[4:], out[4:], sm_quota=37, step_index=[e.step for e in envs[4:]])
    gen.sync()
    gen.destroy()
    assert chunk_rel_err(out.cpu().numpy(), ref) <= TOL[dtype]
    # the planes really differ per layer: feeding layer 0's pair to every layer changes the result
    ref_shared = oracle.actgen(oracle_cfg(w), oracle_weights(wt), [np32(k[:1]) for k in kvs], np.stack([np32(e.noise) for e in envs]),
                               step_index=[e.step for e in envs])
    assert np.abs(ref_shared - ref).max() > 1e-3


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_weight_publication_switches_versions_between_batches(dtype):
    """A new policy version is uploaded while earlier groups are still queued or running: groups
    submitted before the update run with the old weights, groups submitted after it with the new
    ones, and a third update reuses the first set.  Results equal those of fresh handles, bit for bit."""
    w = synth.scaled(synth.WORKLOADS[0], B=10, dtype=dtype, P=(20, 60))
    wA = synth.make_weights(w, 101, random_gains=True)
    wB = synth.make_weights(w, 202, random_gains=True)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    ids = list(range(w.B))
    refs = {}
    for name, wt in (("A", wA), ("B", wB)):
        r = Runner(w, wt, envs)
        refs[name] = stack(r.run([ids]), ids)
        r.close()
    assert not np.array_equal(refs["A"], refs["B"])
    # each version's chunks are the oracle's for that version's weights (and not the other's)
    assert chunk_rel_err(refs["A"], oracle_run(w, wA, envs)) <= TOL[dtype]
    assert chunk_rel_err(refs["B"], oracle_run(w, wB, envs)) <= TOL[dtype]
    assert chunk_rel_err(refs["A"], oracle_run(w, wB, envs)) > 10 * TOL[dtype]
    r = Runner(w, wA, envs, max_inflight_groups=4)
    assert r.gen.weights_version() == 1
    noise = torch.stack([r.noise[e] for e in ids])
    out1, out2 = torch.empty_like(noise), torch.empty_like(noise)
    kv = [r.kv[e] for e in ids]
    r.gen.submit(ids[:6], kv[:6], noise[:6], out1[:6])                 # queued under version 1
    side = torch.cuda.Stream()
    assert r.gen.update_weights(wB, stream=side) == 2                     # launches the queued group, then uploads on a side stream
    r.gen.submit([100 + e for e in ids], kv, noise, out2)                # runs with version 2
    r.gen.sync()
    assert np.array_equal(out1[:6].cpu().numpy(), refs["A"][:6])
    assert np.array_equal(out2.cpu().numpy(), refs["B"])
    assert r.gen.stats()["weights_version"] == 2 and r.gen.weights_version() == 2
    assert r.gen.update_weights(wA) == 3                                  # the first set is overwritten only after its readers
    got = stack(r.run([ids]), ids)
    assert np.array_equal(got, refs["A"]) and r.gen.stats()["weights_version"] == 3
    r.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_rollout_policies_deliver_identical_chunks(dtype):
    """Group-level batching and step-level continuous batching (every Euler step its own submit,
    environments joining mid-chunk) serve the same seeded rollout: every (environment, visit) gets
    the same bits under both policies, and those bits are the oracle's within tolerance."""
    from paper_2609_27547_b200 import rollout_sim as R
    from helpers import oracle_cfg, oracle_weights
    import oracle
    w = synth.scaled(synth.WORKLOADS[0], B=20, dtype=dtype, P=(16, 48), K=4)
    wt = synth.make_weights(w, SEED, random_gains=True)
    a = R.run(w, wt, 20, 3, "chunk", max_group=8, keep_outputs=True)
    b = R.run(w, wt, 20, 3, "step", max_group=8, keep_outputs=True)
    assert a.chunks == b.chunks == 60 and set(a.outputs) == set(b.outputs)
    for k in a.outputs:
        assert torch.equal(a.outputs[k], b.outputs[k]), k
    assert b.submits > a.submits                      # the step policy re-batches every Euler step
    for r in (a, b):
        s = r.summary()
        assert 0 < s["latency_ms"]["p50"] <= s["latency_ms"]["p99"] and 0 < s["generation_busy_frac"] <= 1.0
    # against the oracle for a few (env, visit) pairs
    keys = [(0, 0), (7, 1), (19, 2)]
    envs = [synth.make_env(w, e, SEED) for e, _ in keys]
    noise = np.stack([np32(synth.normal(SEED, "noise_visit%d" % v, e, (w.H, w.A))) for e, v in keys])
    ref = oracle.actgen(oracle_cfg(w), oracle_weights(wt), [np32(e.kv) for e in envs], noise)
    got = np.stack([a.outputs[k].cpu().numpy() for k in keys])
    assert chunk_rel_err(got, ref) <= TOL[dtype]


def test_simulator_latency_model_moments():
    """The synthetic simulator step time: log-normal with mean 40 ms and 99th percentile 60 ms."""
    from paper_2609_27547_b200 import rollout_sim as R
    z = synth.normal(SEED, "sim_latency", 0, (200000,)).double()
    t = torch.exp(R.SIM_MU + R.SIM_SIGMA * z)
    assert abs(float(t.mean()) - 40.0) < 0.2
    assert abs(float(torch.quantile(t, 0.99)) - 60.0) < 0.8


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_chunk_of_five_actions(dtype):
    """The paper's other chunk length ("next 5 or 8 actions"): H = 5, which is neither a power of two nor a
    divisor of the 128-row tile, so environments straddle tile and warp boundaries."""
    w = synth.scaled(synth.WORKLOADS[0], B=53, dtype=dtype, H=5, P=(30, 90), K=3, mixed_steps=True)
    wt, envs = _setup(w)
    ref = oracle_run(w, wt, envs)
    r = Runner(w, wt, envs, max_inflight_groups=3)
    ids = list(range(w.B))
    got = stack(r.run([ids[:20], ids[20:21], ids[21:]], quota=37), ids)
    alone = stack(r.run([[e] for e in ids[:5]]), ids[:5])
    r.close()
    assert chunk_rel_err(got, ref) <= TOL[dtype]
    assert np.array_equal(alone, got[:5])


def test_queue_semantics_flush_streams_and_timing():
    """Queue depth 1 launches at submit (the result is ready after a stream synchronisation, no library
    sync needed); a deeper queue holds groups until flush / a stream or quota change / sync; the
    per-class timing adds up launches and device time."""
    w = synth.scaled(synth.WORKLOADS[0], B=9, P=(20, 40))
    wt, envs = _setup(w)
    ids = list(range(w.B))
    r1 = Runner(w, wt, envs, max_inflight_groups=1)
    base = stack(r1.run([ids]), ids)
    noise = torch.stack([r1.noise[e] for e in ids])
    kv = [r1.kv[e] for e in ids]
    st = torch.cuda.Stream()
    out = torch.zeros_like(noise)
    r1.gen.submit([100 + e for e in ids], kv, noise, out, stream=st)
    st.synchronize()                                   # depth 1: already launched on the caller's stream
    assert np.array_equal(out.cpu().numpy(), base)
    r1.gen.sync()
    r1.close()

    r = Runner(w, wt, envs, max_inflight_groups=4, flags=B.FLAG_TIMING)
    out_a, out_b, out_c = torch.zeros_like(noise), torch.zeros_like(noise), torch.zeros_like(noise)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    r.gen.submit(ids[:4], kv[:4], noise[:4], out_a[:4], stream=s1)          # queued
    s1.synchronize()
    assert float(out_a.abs().sum()) == 0.0 and r.gen.stats()["kernel_launches"] == 0
    r.gen.submit(ids[4:], kv[4:], noise[4:], out_a[4:], stream=s1)          # queued with the first
    r.gen.flush()                                                            # launches both as one batch
    s1.synchronize()
    assert np.array_equal(out_a.cpu().numpy(), base)
    n1 = r.gen.stats()["kernel_launches"]
    assert n1 == w.K * (w.L * 8 + 2)                                        # one batch, not two
    r.gen.sync()                                                             # retire: the ids may be used again
    r.gen.submit(ids[:5], kv[:5], noise[:5], out_b[:5], stream=s1, sm_quota=37)
    r.gen.submit(ids[5:], kv[5:], noise[5:], out_c[5:], stream=s2, sm_quota=37)   # other stream: closes the first batch
    s1.synchronize()
    assert np.array_equal(out_b[:5].cpu().numpy(), base[:5])
    r.gen.sync()
    assert np.array_equal(out_c[5:].cpu().numpy(), base[5:])
    stt = r.gen.stats()
    assert stt["kernel_launches"] == 3 * n1 and stt["groups"] == 4
    cls = stt["classes"]
    assert sum(c["launches"] for c in cls.values()) == stt["kernel_launches"]
    assert cls["gemm"]["launches"] == 3 * w.K * w.L * 6 and cls["gemm"]["ms"] > 0 and cls["gemm"]["flops"] > 0
    assert cls["cross_attn"]["bytes"] > 0 and cls["head"]["launches"] == 3 * w.K
    r.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_two_handles_share_the_gpu_on_disjoint_quotas(dtype):
    """Two handles (two policies co-located on one GPU, as the paper's stages are) run at the same
    time on their own streams under complementary SM quotas; each delivers the bits it delivers alone."""
    w = synth.scaled(synth.WORKLOADS[0], B=12, dtype=dtype, P=(30, 90), mixed_steps=True)
    wA = synth.make_weights(w, 11, random_gains=True)
    wB = synth.make_weights(w, 22, random_gains=True)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    ids = list(range(w.B))
    solo = {}
    for name, wt in (("A", wA), ("B", wB)):
        r = Runner(w, wt, envs)
        solo[name] = stack(r.run([ids], quota=0), ids)
        r.close()
    ra, rb = Runner(w, wA, envs, max_inflight_groups=2), Runner(w, wB, envs, max_inflight_groups=2)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    noise = torch.stack([ra.noise[e] for e in ids])
    outs = {"A": [], "B": []}
    for rep in range(3):                       # interleaved submits, nothing synchronised in between
        for name, r, st, quota in (("A", ra, sa, 100), ("B", rb, sb, 48)):
            out = torch.empty_like(noise)
            half = w.B // 2
            sidx = [envs[e].step for e in ids]
            r.gen.submit([1000 * rep + e for e in ids[:half]], [r.kv[e] for e in ids[:half]], noise[:half], out[:half],
                         sm_quota=quota, stream=st, step_index=sidx[:half])
            r.gen.submit([1000 * rep + e for e in ids[half:]], [r.kv[e] for e in ids[half:]], noise[half:], out[half:],
                         sm_quota=quota, stream=st, step_index=sidx[half:])
            outs[name].append(out)
    ra.gen.sync()
    rb.gen.sync()
    for name in ("A", "B"):
        for out in outs[name]:
            assert np.array_equal(out.cpu().numpy(), solo[name])
    ra.close()
    rb.close()
