"""Host-side checks of the benchmark's workload definitions (no GPU)."""
import bench


def test_paper_shape_reproduces_the_papers_operation_counts():
    # Section 3.3: 0.533 T operations per request with beams (1, 1024, 1024, 1024), 0.446 T with the
    # dynamic schedule (1, 512, 1024, 1024).  d_model and the FFN width are not printed; the shape used
    # here (2048 / 8192) has to land within a few per cent, and the saving must match the paper's ratio.
    fixed = bench.decoder_macs(bench.PAPER_SHAPE, (1, 1024, 1024, 1024))
    dynamic = bench.decoder_macs(bench.PAPER_SHAPE, (1, 512, 1024, 1024))
    assert abs(fixed / 0.533e12 - 1) < 0.05
    assert abs(dynamic / 0.446e12 - 1) < 0.05
    assert abs(dynamic / fixed - 0.446 / 0.533) < 0.005


def test_macs_scale_with_rows_and_context():
    cfg = dict(bench.CFG5)
    base = bench.decoder_macs(cfg)
    wider = bench.decoder_macs(cfg, (1, 4096, 4096, 4096))
    assert 1.9 < wider / base < 2.01                      # row-proportional apart from the per-request K/V projection
    longer = dict(cfg, T_ctx=2 * cfg["T_ctx"])
    assert bench.decoder_macs(longer) > base


def test_bench_workloads_are_consistent():
    for cfg in bench.WORKLOADS.values():
        assert len(cfg["schedule"]) == cfg["L"] and cfg["schedule"][0] == 1
        assert cfg["final_k"] <= cfg["schedule"][-1] * cfg["V"]
        assert cfg["d_model"] % 64 == 0 and (cfg["H"] * cfg["d_h"]) % 64 == 0 and cfg["d_ffn"] % 64 == 0
