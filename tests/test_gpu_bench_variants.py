"""The measurement helpers of include/dynbatch_bench.h: the launch shapes that were measured against the
kept aggregation kernel must produce its results bit for bit (only the data movement differs), and the
read probe must read what it is given."""
import pytest
import torch

from paper_2305_12213_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("K", [2, 4, 8, 16])
@pytest.mark.parametrize("variant,stage", [(binding.DB_BENCH_PERSISTENT, 0), (binding.DB_BENCH_BULK_STAGED, 512),
                                           (binding.DB_BENCH_BULK_STAGED, 1024), (binding.DB_BENCH_BULK_STAGED, 2048)])
def test_rejected_shapes_are_bit_identical_to_the_kept_kernel(K, variant, stage):
    N = 3_000_012                                    # several hundred tiles and a ragged last one
    b = inputs.batch_sizes_uniform(K, 8, 256, 77 + K)
    g = inputs.worker_gradients(K, N, 1e-3, 6000, device=DEV)
    p0, v0 = inputs.normal(N, 0.02, 61, DEV), inputs.normal(N, 0.01, 62, DEV)
    p1, v1, p2, v2 = p0.clone(), v0.clone(), p0.clone(), v0.clone()
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    for _ in range(2):                               # two steps: the second starts from updated state
        binding.aggregate_update(g, b, p1, v1, 0.1, 0.9)
        binding.bench_aggregate_variant(variant, stage, g, b, p2, v2, 0.1, 0.9, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(p1, p2) and torch.equal(v1, v2)


def test_variant_argument_errors():
    N = 4096
    g = inputs.worker_gradients(3, N, 1.0, 6100, device=DEV)
    p, v = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    with pytest.raises(binding.DynbatchError) as ei:                 # K = 3 is not one of the compared sizes
        binding.bench_aggregate_variant(binding.DB_BENCH_PERSISTENT, 0, g, [1, 2, 3], p, v, 0.1, 0.9)
    assert ei.value.status == binding.DB_ERR_UNSUPPORTED
    with pytest.raises(binding.DynbatchError) as ei:                 # unknown stage size
        binding.bench_aggregate_variant(binding.DB_BENCH_BULK_STAGED, 777, g[:2], [1, 2], p, v, 0.1, 0.9)
    assert ei.value.status == binding.DB_ERR_UNSUPPORTED
    with pytest.raises(binding.DynbatchError) as ei:                 # off the 16-byte grid
        binding.bench_aggregate_variant(binding.DB_BENCH_PERSISTENT, 0, [t[1:N - 3] for t in g[:2]], [1, 2],
                                        p[:N - 4], v[:N - 4], 0.1, 0.9)
    assert ei.value.status == binding.DB_ERR_UNSUPPORTED
    assert not p.any().item() and not v.any().item()


def test_read_probe_reads_every_byte_it_is_given():
    n = (1 << 22) + 16                                # a ragged last CTA
    src = torch.zeros(n, dtype=torch.uint8, device=DEV)
    sink = torch.empty(binding.bench_read_probe_sink_bytes(n), dtype=torch.uint8, device=DEV)
    binding.bench_read_probe(src, sink)
    torch.cuda.synchronize()
    zero = sink.clone()
    assert not zero.any().item()                      # zeros in, zero checksums out
    for pos in (0, 12345 * 16 + 3, n - 1):            # one byte anywhere changes some checksum
        src.zero_()
        src[pos] = 1
        binding.bench_read_probe(src, sink)
        torch.cuda.synchronize()
        assert sink.any().item(), pos
    with pytest.raises(binding.DynbatchError):
        binding.bench_read_probe(src[:100], sink)     # not a multiple of 16 bytes


def test_a_wait_that_never_ends_gives_up_and_reports():
    """The tensor-core kernels bound every mbarrier wait and report a time-out through a status word.
    Here the wait is made to run out on purpose (nothing ever arrives), with a short limit: the kernel
    returns normally, the code is in the status word, and the device goes on working."""
    import time
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    binding.bench_wait_timeout(status, 77, 50_000_000)          # 50 ms
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    assert int(status.item()) == 77
    assert 0.04 < waited < 1.5
    # the first code stays: a second time-out does not overwrite it
    binding.bench_wait_timeout(status, 78, 1_000_000)
    torch.cuda.synchronize()
    assert int(status.item()) == 77
    # the context is intact: an ordinary step runs and is right
    N = 4096
    g = [torch.ones(N, device=DEV) for _ in range(2)]
    p, v = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    binding.aggregate_update(g, [1, 1], p, v, 0.5, 0.0)
    torch.cuda.synchronize()
    assert torch.equal(v, torch.ones(N, device=DEV))
    with pytest.raises(binding.DynbatchError):
        binding.bench_wait_timeout(status, 0, 1000)
    with pytest.raises(binding.DynbatchError):
        binding.bench_wait_timeout(status, 5, 3_000_000_000)     # beyond the kernels' own 2 s limit
