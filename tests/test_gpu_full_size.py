"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times (sr_rollout_run
with CUDA graphs of 16 frames, tensor cores where they apply).  The oracle evaluates a few whole
sequences of the batch (sequences are independent, so those samples are exact); output sequence and
final states of every node are compared.  The benchmarked runs themselves are compared in full length on one
sequence each: c5 (64 x 64 images, all 128 frames; streaming and one hybrid) and c4 sequential (all 64 frames)."""
import pytest

from tests import parity
from workloads import graphs

pytestmark = pytest.mark.gpu


def test_c2_full_size_all_patterns():
    g = graphs.build("c2")
    for p in g.patterns:
        parity.check_run(g, p, graph_frames=16, samples=[0, 31, 63], expect_resident=2)      # the resident kernel
        parity.check_run(g, p, graph_frames=16, samples=[0, 31, 63], resident=False)         # per-frame launches


def test_c3_full_size_all_patterns():
    g = graphs.build("c3")
    for p in g.patterns:
        parity.check_run(g, p, graph_frames=16, samples=[0, 255])


def test_c4_full_size_streaming():
    g = graphs.build("c4")
    parity.check_run(g, "streaming", graph_frames=16, samples=[0, 127])


def test_c4_full_size_sequential_all_frames():
    g = graphs.build("c4")
    parity.check_run(g, "sequential", graph_frames=16, samples=[64])


def test_c5_full_size_fewer_frames():
    g = graphs.build("c5", frames=10)
    parity.check_run(g, "streaming", graph_frames=4, samples=[0, 31])
    g2 = graphs.build("c5", frames=3)
    for p in ("sequential", "hybrid0", "hybrid1", "hybrid2"):
        parity.check_run(g2, p, graph_frames=0, samples=[17])


@pytest.mark.parametrize("pattern", ["streaming", "hybrid1"])
def test_c5_full_size_all_128_frames(pattern):
    # the run bench.py times: batch 32, 64 x 64 images, 128 frames, CUDA graphs of 16 frames; the oracle follows one
    # whole sequence (about 0.7 T multiply-adds), which is exact because sequences are independent
    g = graphs.build("c5")
    parity.check_run(g, pattern, graph_frames=16, samples=[13])


def test_c5_all_128_frames_reduced_images():
    # recurrent edges over 128 frames with states re-rounded to bf16 every frame: the drift stays in tolerance
    g = graphs.build("c5", size=16, batch=8)
    for p in ("streaming", "hybrid1"):
        parity.check_run(g, p, graph_frames=16, samples=[0, 7])


@pytest.mark.parametrize("name,options", [("c3", dict(tc_fuse=0, tc_lists=1)), ("c4", dict(tc_fuse=0, tc_lists=1, stem_ring=0)),
                                          ("c4", dict(stem_ring=2))])
def test_full_size_with_the_optional_paths_switched(name, options):
    # every node on its own, per-CTA work lists only, staged boxes in / out of the weight ring: same results
    g = graphs.build(name, frames=6)
    parity.check_run(g, "streaming", graph_frames=0, samples=[1], **options)
