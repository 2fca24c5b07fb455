"""The MMA-issue-only measurement kernel (falqon_tensor_ceiling): it must finish cleanly, account for its work, really
run the products (zero operands give zero accumulators, pseudo-random ones do not, the same seed gives the same
sums) and take time in proportion to the work it is given."""
import pytest
import torch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def fq():
    from paper_2510_24061_b200 import binding
    return binding


def _sink(fq):
    return torch.full((4 * fq.tensor_ceiling_ctas(),), float("nan"), dtype=torch.float32, device=DEV)


def test_accounting_and_clean_exit(fq):
    ctas = fq.tensor_ceiling_ctas()
    assert ctas % 2 == 0 and ctas >= 2
    for kblocks in (1, 3, 4, 33, 130):           # fewer k-blocks than operand slots, and across accumulator changes
        sink = _sink(fq)
        flops = fq.tensor_ceiling(kblocks, 5, True, sink)
        assert flops == (ctas // 2) * kblocks * 4 * 2 * 256 * 256 * 32
        torch.cuda.synchronize()
        assert fq.last_device_status() == 0
        assert bool(torch.isfinite(sink).all())
    with pytest.raises(fq.FalqonError):
        fq.tensor_ceiling(0)
    with pytest.raises(fq.FalqonError):
        fq.tensor_ceiling((1 << 20) + 1)


def test_the_products_are_computed(fq):
    zero, a, b, c = _sink(fq), _sink(fq), _sink(fq), _sink(fq)
    fq.tensor_ceiling(40, 9, False, zero)
    fq.tensor_ceiling(40, 9, True, a)
    fq.tensor_ceiling(40, 9, True, b)
    fq.tensor_ceiling(40, 10, True, c)
    torch.cuda.synchronize()
    assert not bool(zero.any())
    assert bool((a != 0).all()) and torch.equal(a, b) and not torch.equal(a, c)
    d = _sink(fq)
    fq.tensor_ceiling(40, 9, 2, d)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(d).all()) and bool((d != 0).any()) and not torch.equal(a, d)
    assert fq.last_device_status() == 0


def test_time_is_proportional_to_the_work_and_the_rate_is_plausible(fq):
    def run(kblocks):
        for _ in range(2):
            fq.tensor_ceiling(kblocks, 1, True)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        flops = 0.0
        for _ in range(5):
            flops += fq.tensor_ceiling(kblocks, 1, True)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e-3, flops
    t1, f1 = run(4000)
    t2, f2 = run(16000)
    assert 2.5 < t2 / t1 < 6.0, (t1, t2)        # four times the work; the first, shorter run may see a slower clock
    tflops = f2 / t2 / 1e12
    print(f"[tensor ceiling] {tflops:.0f} TFLOP/s over {t2 * 1e3:.1f} ms")
    assert 1000.0 < tflops < 4500.0 * 1.05          # above the nominal peak the kernel would not be doing the work
    assert fq.last_device_status() == 0


def test_with_the_operand_stream(fq):
    """The producer/consumer form (operands streamed from a buffer while the MMAs run) finishes cleanly for k-block counts
    around the ring size, and the MMAs then see the buffer's contents: a buffer of zeros gives zero sums whatever the fill."""
    src = torch.zeros(1 << 20, dtype=torch.uint8, device=DEV)
    for kblocks in (1, 5, 6, 7, 40, 1000):
        sink = _sink(fq)
        fq.tensor_ceiling(kblocks, 3, 1, sink, src)
        torch.cuda.synchronize()
        assert fq.last_device_status() == 0
        assert bool(torch.isfinite(sink).all())
        if kblocks >= 40:
            assert not bool(sink.any())      # the last accumulation ran entirely on streamed (zero) operands
    with pytest.raises(fq.FalqonError):
        fq.tensor_ceiling(8, 3, 1, None, src[:16384])
