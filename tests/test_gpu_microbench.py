"""const_microbench: the machine-limit micro-benchmarks that the benchmark rates the fused kernels against.
Checked here: argument validation, that every kind runs and reports the work it states in the header, and that
the figures land in the range the hardware's unit counts allow (a kernel the compiler emptied, or a timer around
nothing, would report far more)."""
import numpy as np
import pytest
import torch

import paper_2401_04836_b200 as cb

pytestmark = pytest.mark.gpu


def _sms():
    return torch.cuda.get_device_properties(0).multi_processor_count


def test_fma_and_matrix_peaks_are_plausible():
    clock_hz = 2.1e9                                              # above any SM clock of the part
    for kind, per_sm_clk in ((cb.BENCH_FP32_FMA, 128 * 2), (cb.BENCH_FP64_FMA, 64 * 2), (cb.BENCH_FP64_MMA, 64 * 2)):
        ms, flop = cb.const_microbench(kind, repeats=3)
        tflops = flop / (ms * 1e-3) / 1e12
        ceiling = _sms() * per_sm_clk * clock_hz / 1e12
        assert ms > 0 and flop > 0
        assert 0.4 * ceiling < tflops < 1.02 * ceiling, (kind, tflops, ceiling)
    ms, flop = cb.const_microbench(cb.BENCH_TF32_MMA, repeats=3)
    tflops = flop / (ms * 1e-3) / 1e12
    assert 300.0 < tflops < 1300.0, tflops                        # nominal dense tf32: about 1100 TFLOP/s


def test_row_gather_counts_the_rows_it_reads():
    rng = np.random.default_rng(5)
    table_rows, n = 50_000, 4_000_000
    rows = torch.from_numpy(rng.integers(0, table_rows, n, dtype=np.int32)).cuda()
    for rank in (8, 16, 32):
        ms, nbytes = cb.const_microbench(cb.BENCH_ROW_GATHER, rows, table_rows=table_rows, rank=rank, repeats=3)
        assert nbytes == n * rank * 4
        assert 0 < ms and nbytes / (ms * 1e-3) < 40e12            # below any on-chip bandwidth of the part


def test_argument_checks():
    rows = torch.zeros(16, dtype=torch.int32, device="cuda")
    for kwargs in (dict(kind=7), dict(kind=-1), dict(kind=cb.BENCH_FP32_FMA, repeats=0),
                   dict(kind=cb.BENCH_ROW_GATHER, rows=None, table_rows=4, rank=8),
                   dict(kind=cb.BENCH_ROW_GATHER, rows=rows, table_rows=4, rank=12),
                   dict(kind=cb.BENCH_ROW_GATHER, rows=rows, table_rows=0, rank=8)):
        with pytest.raises(cb.ConstError) as e:
            cb.const_microbench(**kwargs)
        assert e.value.status == 1
