"""GPU parity of db_aggregate_update_ex against the fp64 oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import BF16_TOL, FP32_TOL, f64, host_grad, rel_err, sample_indices
from paper_2305_12213_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _workspace(K, N):
    return torch.empty(binding.aggregate_workspace_bytes(K, N), dtype=torch.uint8, device=DEV)


def _run_both(grads, b, p0, v0, lr, mu, norm=True):
    """GPU call and oracle call from the same stored state; returns (gpu p, v, sq), (ref p, v, sq)."""
    K, N = len(grads), p0.numel()
    p, v = p0.clone(), v0.clone()
    sq = torch.zeros(1, dtype=torch.float64, device=DEV) if norm else None
    ws = _workspace(K, N) if norm else None
    binding.aggregate_update(grads, b, p, v, lr, mu, sq, ws)
    torch.cuda.synchronize()
    rp, rv = f64(p0), f64(v0)
    _, rsq = oracle.aggregate_update([host_grad(g) for g in grads], b, rp, rv,
                                     float(np.float32(lr)), float(np.float32(mu)))
    return (p, v, None if sq is None else float(sq.item())), (rp, rv, rsq)


def _assert_close(gpu, ref, tol=FP32_TOL):
    (p, v, sq), (rp, rv, rsq) = gpu, ref
    assert rel_err(f64(p), rp) <= tol
    assert rel_err(f64(v), rv) <= tol
    if sq is not None:
        assert abs(sq - rsq) <= tol * max(rsq, 1e-300)


@pytest.mark.parametrize("N", [1, 3, 4, 5, 7, 8, 9, 1023, 1024, 1025, 4099, 70001, 300000])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_sizes_and_ragged_tails(N, dtype):
    K = 3
    grads = inputs.worker_gradients(K, N, 1.0, 10, device=DEV, dtype=dtype)
    p0 = inputs.normal(N, 0.02, 1, DEV)
    v0 = inputs.normal(N, 0.5, 2, DEV)
    _assert_close(*_run_both(grads, [16, 32, 80], p0, v0, 0.1, 0.9))


@pytest.mark.parametrize("K", [1, 2, 3, 4, 5, 7, 8, 9, 15, 16, 17, 24, 31, 32, 33, 64])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_worker_counts(K, dtype):
    N = 50_003
    grads = inputs.worker_gradients(K, N, 1.0, 20, device=DEV, dtype=dtype)
    b = inputs.batch_sizes_uniform(K, 8, 256, K)
    p0 = inputs.normal(N, 0.02, 3, DEV)
    v0 = inputs.normal(N, 0.5, 4, DEV)
    _assert_close(*_run_both(grads, b, p0, v0, 0.05, 0.9))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("offset", [0, 1, 2, 3, 5])
def test_shifted_but_congruent_pointers_take_the_vector_path(dtype, offset):
    """All buffers start `offset` elements into 16-byte aligned allocations of their own type."""
    N, K = 10_007, 4
    esz = 4 if dtype == torch.float32 else 2
    # shift gradients so that they stay congruent with the fp32 state: same element offset
    goff = offset if dtype == torch.float32 else offset
    backing = [inputs.normal(N + 16, 1.0, 30 + k, DEV, dtype) for k in range(K)]
    grads = [t[goff:goff + N] for t in backing]
    pb, vb = inputs.normal(N + 16, 0.02, 5, DEV), inputs.normal(N + 16, 0.5, 6, DEV)
    p0, v0 = pb[offset:offset + N], vb[offset:offset + N]
    assert all(g.data_ptr() % esz == 0 for g in grads)
    gpu, ref = _run_both(grads, [24, 40, 64, 128], p0, v0, 0.1, 0.9)
    _assert_close(gpu, ref)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_incongruent_pointers_fall_back_and_agree_bitwise(dtype):
    """Mixed offsets force the element-wise kernel; p and v must equal the vector path bit for bit."""
    N, K = 20_011, 5
    b = [3, 9, 18, 5, 12]
    backing = [inputs.normal(N + 16, 1.0, 40 + k, DEV, dtype) for k in range(K)]
    aligned = [t[:N].clone() for t in backing]
    shifted = []
    for k, t in enumerate(backing):
        s = torch.empty(N + 16, dtype=dtype, device=DEV)
        s[k % 4 + 1:k % 4 + 1 + N] = t[:N]
        shifted.append(s[k % 4 + 1:k % 4 + 1 + N])
    p0, v0 = inputs.normal(N, 0.02, 7, DEV), inputs.normal(N, 0.5, 8, DEV)
    (p1, v1, s1), ref = _run_both(aligned, b, p0, v0, 0.1, 0.9)
    (p2, v2, s2), _ = _run_both(shifted, b, p0, v0, 0.1, 0.9)
    _assert_close((p2, v2, s2), ref)
    assert torch.equal(p1, p2) and torch.equal(v1, v2)


def test_bf16_gradients_equal_their_fp32_widening_bitwise():
    N, K = 123_457, 6
    g16 = inputs.worker_gradients(K, N, 1e-3, 50, device=DEV, dtype=torch.bfloat16)
    g32 = [g.float() for g in g16]
    b = [5, 9, 2, 30, 11, 7]
    p0, v0 = inputs.normal(N, 0.02, 9, DEV), inputs.normal(N, 0.1, 10, DEV)
    (pa, va, sa), _ = _run_both(g16, b, p0, v0, 0.05, 0.9)
    (pb, vb, sb), _ = _run_both(g32, b, p0, v0, 0.05, 0.9)
    assert torch.equal(pa, pb) and torch.equal(va, vb)
    assert abs(sa - sb) <= 1e-7 * sb       # the norm's fp32 lane grouping differs (8 vs 4 lanes)


def test_bf16_against_unrounded_gradients():
    """Storing gradients as bf16 (8 significant bits, unit roundoff 2^-8) perturbs each g_k[j] by at
    most 2^-8 |g_k[j]|, hence the aggregate by at most 2^-8 sum_k lambda_k |g_k[j]|: within 1e-2 of
    the oracle fed the unrounded fp32 gradients, relative to that aggregated magnitude."""
    N, K = 200_000, 16
    g32 = inputs.worker_gradients(K, N, 1e-3, 60, device=DEV)
    g16 = [g.to(torch.bfloat16) for g in g32]
    b = inputs.batch_sizes_uniform(K, 8, 256, 3)
    p0, v0 = inputs.normal(N, 0.02, 11, DEV), torch.zeros(N, device=DEV)
    p, v = p0.clone(), v0.clone()
    binding.aggregate_update(g16, b, p, v, 0.05, 0.9)
    torch.cuda.synchronize()
    rp, rv = f64(p0), f64(v0)
    oracle.aggregate_update([host_grad(g) for g in g32], b, rp, rv, float(np.float32(0.05)), float(np.float32(0.9)))
    lam = oracle.weights(b)
    scale = sum(l * np.abs(f64(g)) for l, g in zip(lam, g32))
    assert np.max(np.abs(f64(v) - rv) / scale) <= BF16_TOL          # v0 = 0, so v is the aggregate
    assert rel_err(f64(p), rp) <= BF16_TOL
    # and the rms-floored metric stays of the same order (reported, looser: cancellation in the sum)
    assert rel_err(f64(v), rv) <= 2.5 * BF16_TOL


def test_zero_batch_worker_is_never_read():
    N = 4096
    g = inputs.worker_gradients(3, N, 1.0, 70, device=DEV)
    g[1].fill_(float("nan"))
    p0, v0 = inputs.normal(N, 0.02, 12, DEV), inputs.normal(N, 0.5, 13, DEV)
    gpu, ref = _run_both(g, [5, 0, 9], p0, v0, 0.1, 0.9)
    _assert_close(gpu, ref)
    assert torch.isfinite(gpu[0]).all()


def test_equal_batches_are_the_plain_mean_and_k1_is_identity():
    N = 8192
    g = inputs.worker_gradients(4, N, 1.0, 80, device=DEV)
    p, v = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    binding.aggregate_update(g, [32] * 4, p, v, 1.0, 0.0)
    mean = torch.stack(g).double().mean(0)
    assert rel_err(f64(v), mean.cpu().numpy()) <= 1e-6
    assert torch.equal(p, -v)
    p.zero_(); v.zero_()
    binding.aggregate_update(g[:1], [7], p, v, 1.0, 0.0)
    assert torch.equal(v, g[0])


@pytest.mark.parametrize("K", [2, 4, 8, 16])
def test_equal_batches_with_k_a_power_of_two_are_the_fp32_mean_bit_for_bit(K):
    """lambda = 1/K is then exact in fp32 and lambda * g_k exact too, so the kernel's chain
    acc = fma(lambda, g_k, acc), k ascending from zero, is the left-to-right fp32 sum of the scaled gradients."""
    N = 70_001
    g = inputs.worker_gradients(K, N, 1.0, 81 + K, device=DEV)
    p, v = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    binding.aggregate_update(g, [24] * K, p, v, 1.0, 0.0)
    acc = torch.zeros(N, device=DEV)
    for gk in g:
        acc = acc + gk * (1.0 / K)
    assert torch.equal(v, acc) and torch.equal(p, -acc)


def test_scaling_every_batch_size_changes_at_most_the_last_bit():
    """b -> c b leaves the weights b_k / sum b unchanged as real numbers; formed in fp64 and rounded to fp32
    they can differ in the last place at most, and so can the aggregate."""
    N, K = 50_003, 5
    g = inputs.worker_gradients(K, N, 1.0, 87, device=DEV)
    b = [7, 13, 32, 58, 6]
    outs = []
    for c in (1, 3, 1000):
        p, v = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
        binding.aggregate_update(g, [c * x for x in b], p, v, 1.0, 0.0)
        outs.append(v)
    scale = torch.stack([x.abs() for x in g]).amax(0)          # an ulp of the largest term bounds the change
    for o in outs[1:]:
        assert bool(((o - outs[0]).abs() <= K * scale * 2.0 ** -23).all())


def test_norm_of_ones_is_exactly_N():
    N = 1_000_003
    ones = [torch.ones(N, device=DEV) for _ in range(4)]
    p, v = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    sq = torch.zeros(1, dtype=torch.float64, device=DEV)
    binding.aggregate_update(ones, [64] * 4, p, v, 0.1, 0.9, sq, _workspace(4, N))
    assert float(sq.item()) == float(N)


def test_overlapping_steps_on_two_streams_keep_their_norms_apart():
    """Two streams run norm-carrying steps at the same time, each with its own workspace.  Every norm
    must be its own problem's."""
    K, calls = 2, 300
    sizes = (300_001, 777_777)
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    state = []
    for i, N in enumerate(sizes):
        g = [torch.full((N,), float(i + 1), device=DEV) for _ in range(K)]
        state.append((g, torch.zeros(N, device=DEV), torch.zeros(N, device=DEV),
                      torch.zeros(calls, dtype=torch.float64, device=DEV), _workspace(K, N)))
    torch.cuda.synchronize()
    for c in range(calls):
        for i, s in enumerate(streams):
            g, p, v, sq, ws = state[i]
            binding.aggregate_update(g, [3, 5], p, v, 0.0, 0.0, sq[c:c + 1], ws, s)
    torch.cuda.synchronize()
    for i, N in enumerate(sizes):
        want = float(N) * (i + 1) ** 2
        got = state[i][3].cpu().numpy()
        assert (got == want).all(), (i, got[got != want][:5], want)


def test_runs_are_bit_identical_and_norm_flag_does_not_change_the_update():
    N, K = 3_000_017, 8
    g = inputs.worker_gradients(K, N, 1e-3, 90, device=DEV)
    b = [32] * 4 + [58] * 2 + [6] * 2
    p0, v0 = inputs.normal(N, 0.02, 14, DEV), inputs.normal(N, 0.01, 15, DEV)
    outs = [_run_both(g, b, p0, v0, 0.1, 0.9, norm=True)[0] for _ in range(3)]
    for o in outs[1:]:
        assert torch.equal(o[0], outs[0][0]) and torch.equal(o[1], outs[0][1]) and o[2] == outs[0][2]
    plain = _run_both(g, b, p0, v0, 0.1, 0.9, norm=False)[0]
    assert torch.equal(plain[0], outs[0][0]) and torch.equal(plain[1], outs[0][1])


def test_short_form_matches_full_form():
    N, K = 65_537, 3
    g = inputs.worker_gradients(K, N, 1.0, 95, device=DEV)
    p0, v0 = inputs.normal(N, 0.02, 16, DEV), inputs.normal(N, 0.5, 17, DEV)
    p1, v1, p2, v2 = p0.clone(), v0.clone(), p0.clone(), v0.clone()
    import ctypes
    table = (ctypes.c_void_p * K)(*[t.data_ptr() for t in g])
    bb = (ctypes.c_int32 * K)(16, 32, 80)
    torch.cuda.synchronize()
    with torch.cuda.stream(torch.cuda.default_stream()):
        st = binding.lib().db_aggregate_update(ctypes.cast(table, ctypes.c_void_p), ctypes.cast(bb, ctypes.c_void_p),
                                               K, N, p1.data_ptr(), v1.data_ptr(), 0.1, 0.9)
    assert st == binding.DB_OK
    torch.cuda.synchronize()
    binding.aggregate_update(g, [16, 32, 80], p2, v2, 0.1, 0.9)
    torch.cuda.synchronize()
    assert torch.equal(p1, p2) and torch.equal(v1, v2)


def test_prepared_step_is_the_same_call():
    """binding.AggregateStep marshals the tensors once; every run must be the plain call's result."""
    N, K = 300_007, 5
    g = inputs.worker_gradients(K, N, 1e-3, 97, device=DEV, dtype=torch.bfloat16)
    p0, v0 = inputs.normal(N, 0.02, 18, DEV), inputs.normal(N, 0.01, 19, DEV)
    p1, v1, p2, v2 = p0.clone(), v0.clone(), p0.clone(), v0.clone()
    sq1 = torch.zeros(1, dtype=torch.float64, device=DEV)
    sq2 = torch.zeros(1, dtype=torch.float64, device=DEV)
    ws1, ws2 = _workspace(K, N), _workspace(K, N)
    step = binding.AggregateStep(g, p2, v2, sq2, ws2)
    for b in ([3, 9, 0, 18, 5], [7, 7, 7, 7, 7]):
        binding.aggregate_update(g, b, p1, v1, 0.1, 0.9, sq1, ws1)
        step.run(b, 0.1, 0.9)
        torch.cuda.synchronize()
        assert torch.equal(p1, p2) and torch.equal(v1, v2) and float(sq1.item()) == float(sq2.item())
    with pytest.raises(ValueError):
        step.run([1, 2], 0.1, 0.9)
    with pytest.raises(binding.DynbatchError):
        step.run([0] * K, 0.1, 0.9)


def test_on_a_side_stream():
    N, K = 500_000, 4
    g = inputs.worker_gradients(K, N, 1.0, 96, device=DEV)
    p0, v0 = inputs.normal(N, 0.02, 18, DEV), inputs.normal(N, 0.5, 19, DEV)
    s = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        gpu, ref = _run_both(g, [1, 2, 3, 4], p0, v0, 0.1, 0.9)
    _assert_close(gpu, ref)


def test_back_to_back_steps_between_foreign_kernels_without_synchronising():
    """Steps are scheduled under their predecessor in the stream (programmatic dependent launch) and
    wait for it themselves.  Seven steps, each right behind a torch kernel that writes that step's
    gradients, alternately with and without the norm, nothing synchronised until the end: the state
    must be what the oracle gets from the same gradients in the same order."""
    N, K, steps = 2_000_003, 5, 7
    b = [7, 1, 0, 30, 12]
    base = [inputs.worker_gradients(K, N, 1e-3, 700 + 10 * it, device=DEV) for it in range(steps)]
    work = [[torch.empty_like(t) for t in base[0]] for _ in range(2)]
    p = inputs.normal(N, 0.02, 41, DEV)
    v = inputs.normal(N, 0.01, 42, DEV)
    rp, rv = f64(p), f64(v)
    sq = torch.zeros(steps, dtype=torch.float64, device=DEV)
    ws = _workspace(K, N)
    torch.cuda.synchronize()
    for it in range(steps):
        g = work[it % 2]
        for k in range(K):
            torch.mul(base[it][k], 2.0, out=g[k])          # a foreign kernel produces this step's gradients
        binding.aggregate_update(g, b, p, v, 0.05, 0.9, sq[it:it + 1] if it % 2 == 0 else None,
                                 ws if it % 2 == 0 else None)
    torch.cuda.synchronize()
    ref_sq = []
    for it in range(steps):
        _, s = oracle.aggregate_update([host_grad(t) * np.float32(2.0) for t in base[it]], b, rp, rv,
                                       float(np.float32(0.05)), float(np.float32(0.9)))
        ref_sq.append(s)
    assert rel_err(f64(p), rp) <= FP32_TOL and rel_err(f64(v), rv) <= FP32_TOL
    got = sq.cpu().numpy()
    for it in range(0, steps, 2):
        assert abs(got[it] - ref_sq[it]) <= FP32_TOL * ref_sq[it]


# ------------------------------------------------------------------ the named configurations
def _iterate(K, N, dtype, g_std, b0, X_of_iter, kp, lr, mu, iters, seed, full_at, sample=1 << 18):
    """Controller step + aggregate/update per iteration with fresh gradients; the oracle is run
    teacher-forced (from the GPU's stored state) and free-running (its own fp64 state), on all
    elements at the iterations in `full_at` and on a fixed index sample at every iteration."""
    p = inputs.normal(N, 0.02, seed, DEV)
    v = torch.zeros(N, device=DEV)
    idx_np = sample_indices(N, sample)
    idx = torch.from_numpy(idx_np).to(DEV)
    free_p, free_v = f64(p[idx]), f64(v[idx])
    sq = torch.zeros(1, dtype=torch.float64, device=DEV)
    ws = _workspace(K, N)
    b_gpu, b_ref = list(b0), np.array(b0, dtype=np.int32)
    lr64, mu64 = float(np.float32(lr)), float(np.float32(mu))
    worst = {"forced": 0.0, "free": 0.0, "sq": 0.0}
    for it in range(iters):
        X = X_of_iter(it)
        b_gpu = binding.controller_step(b_gpu, X, kp)
        b_ref = oracle.controller_step(b_ref, X, kp)
        assert b_gpu == b_ref.tolist(), f"controller diverged at iteration {it}"
        grads = inputs.worker_gradients(K, N, g_std, seed + 1, it, DEV, dtype)
        full = it in full_at
        if full:
            p_before, v_before = f64(p), f64(v)
        sp_before, sv_before = f64(p[idx]), f64(v[idx])
        binding.aggregate_update(grads, b_gpu, p, v, lr, mu, sq, ws)
        torch.cuda.synchronize()
        hg = [host_grad(g[idx]) for g in grads]
        # teacher-forced, sampled
        oracle.aggregate_update(hg, b_ref, sp_before, sv_before, lr64, mu64)
        worst["forced"] = max(worst["forced"], rel_err(f64(p[idx]), sp_before), rel_err(f64(v[idx]), sv_before))
        # free-running, sampled
        oracle.aggregate_update(hg, b_ref, free_p, free_v, lr64, mu64)
        worst["free"] = max(worst["free"], rel_err(f64(p[idx]), free_p), rel_err(f64(v[idx]), free_v))
        if full:
            _, rsq = oracle.aggregate_update([host_grad(g) for g in grads], b_ref, p_before, v_before, lr64, mu64)
            worst["forced"] = max(worst["forced"], rel_err(f64(p), p_before), rel_err(f64(v), v_before))
            worst["sq"] = max(worst["sq"], abs(float(sq.item()) - rsq) / rsq)
        del grads
    return b_gpu, worst


def test_config_small_three_workers_ten_iterations():
    """K=3, N=2^20 fp32, b={16,32,80}, throughputs {1,2,5}, kp=0.5: a controller fixed point."""
    b, worst = _iterate(3, 1 << 20, torch.float32, 1.0, [16, 32, 80], lambda it: [1.0, 2.0, 5.0], 0.5,
                        0.1, 0.9, 10, 1234, full_at=set(range(10)), sample=1 << 20)
    assert b == [16, 32, 80]
    assert worst["forced"] <= FP32_TOL and worst["free"] <= FP32_TOL and worst["sq"] <= FP32_TOL


def test_config_resnet50_eight_workers_hundred_iterations():
    """161 ResNet-50 tensors in one arena (25,557,032 fp32), 4 fast + 4 slow workers, global batch 256."""
    N = inputs.RESNET50_N
    assert inputs.tensor_offsets(inputs.resnet50_tensor_shapes())[-1] == N
    X = [10.0] * 4 + [1.0] * 4
    b, worst = _iterate(8, N, torch.float32, 1e-3, [32] * 8, lambda it: X, 1.0, 0.1, 0.9, 100, 2000,
                        full_at={0, 1, 99})
    assert b == [58] * 4 + [6] * 4
    assert worst["forced"] <= FP32_TOL and worst["free"] <= FP32_TOL and worst["sq"] <= FP32_TOL


def test_resnet50_per_tensor_calls_equal_the_flat_call():
    N = inputs.RESNET50_N
    offs = inputs.tensor_offsets(inputs.resnet50_tensor_shapes())
    K, b = 8, [58] * 4 + [6] * 4
    g = inputs.worker_gradients(K, N, 1e-3, 2100, device=DEV)
    p0, v0 = inputs.normal(N, 0.02, 21, DEV), inputs.normal(N, 0.01, 22, DEV)
    p1, v1, p2, v2 = p0.clone(), v0.clone(), p0.clone(), v0.clone()
    binding.aggregate_update(g, b, p1, v1, 0.1, 0.9)
    for s, e in zip(offs[:-1], offs[1:]):
        binding.aggregate_update([t[s:e] for t in g], b, p2[s:e], v2[s:e], 0.1, 0.9)
    torch.cuda.synchronize()
    assert torch.equal(p1, p2) and torch.equal(v1, v2)


def test_config_bert_base_sixteen_workers_bf16():
    """199 BERT-base tensors (109,482,240 params), bf16 gradients, lognormal throughputs, worker 3
    halves its throughput at iteration 50; 200 iterations, global batch 512."""
    N = inputs.BERT_BASE_N
    assert inputs.tensor_offsets(inputs.bert_base_tensor_shapes())[-1] == N
    X0 = inputs.lognormal_throughputs(16, 0.5, 4242)

    def X_of(it):
        X = list(X0)
        if it >= 50:
            X[3] *= 0.5
        return X

    b, worst = _iterate(16, N, torch.bfloat16, 1e-3, [32] * 16, X_of, 1.0, 0.05, 0.9, 200, 3000,
                        full_at={0, 1, 2, 49, 50, 51, 52, 199}, sample=1 << 20)
    assert sum(b) == 512
    want = 512 * np.array(X_of(199)) / sum(X_of(199))
    assert np.abs(np.array(b) - want).max() <= 1.0
    assert worst["forced"] <= FP32_TOL and worst["free"] <= FP32_TOL and worst["sq"] <= FP32_TOL


SWEEP = [(n, k) for n in (1 << 20, 1 << 22, 1 << 24, 1 << 26, 1 << 28) for k in (2, 4, 8, 16, 32)
         if n * k <= (1 << 33)]


@pytest.mark.parametrize("N,K", SWEEP)
def test_bandwidth_sweep_points_on_sampled_outputs(N, K):
    """Every (N, K) of the bandwidth sweep, in the launch the benchmark times, checked on a sample."""
    b = inputs.batch_sizes_uniform(K, 8, 256, 5000 + K)
    grads = inputs.worker_gradients(K, N, 1.0, 5100, device=DEV)
    p = inputs.normal(N, 0.02, 23, DEV)
    v = inputs.normal(N, 0.5, 24, DEV)
    idx_np = sample_indices(N, 1 << 16)
    idx = torch.from_numpy(idx_np).to(DEV)
    rp, rv = f64(p[idx]), f64(v[idx])
    sq = torch.zeros(1, dtype=torch.float64, device=DEV)
    binding.aggregate_update(grads, b, p, v, 0.1, 0.9, sq, _workspace(K, N))
    torch.cuda.synchronize()
    g, _ = oracle.aggregate_update([host_grad(t[idx]) for t in grads], b, rp, rv,
                                   float(np.float32(0.1)), float(np.float32(0.9)), want_g=True)
    assert rel_err(f64(p[idx]), rp) <= FP32_TOL and rel_err(f64(v[idx]), rv) <= FP32_TOL
    # the norm is a property of all N elements: sum of squares of a weighted sum of N(0,1) draws
    lam = np.array(b, dtype=np.float64) / sum(b)
    expect = N * float((lam ** 2).sum())
    assert abs(float(sq.item()) / expect - 1.0) < 6.0 / np.sqrt(N) + 1e-3
    del grads
