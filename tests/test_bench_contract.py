"""CPU checks of the benchmark's contract: the default workload is the largest single-GPU configuration, and the CUDA
arm and the reference arm describe a workload with the same `config` object (so that their lines are comparable)."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
import matkv_inputs as mi  # noqa: E402


def test_default_workload_is_the_headline_configuration():
    args = bench.parse_args([])
    assert args.workload == bench.HEADLINE == "cfg4" and args.gpus == 1 and args.impl == "matkv"
    w = mi.workload(args.workload)
    # the largest configuration that fits one GPU: 128 chunks of 640 MiB
    assert w.pool_chunks * w.chunk_bytes == 128 * 80 * 2 * 8 * 2048 * 128 * 2
    assert all(mi.workload(n).pool_chunks * mi.workload(n).chunk_bytes <= w.pool_chunks * w.chunk_bytes for n in ("cfg1", "cfg2", "cfg3", "cfg5"))


def test_both_arms_describe_a_workload_with_the_same_config():
    for name in ("cfg2", "cfg4"):
        w = mi.workload(name)
        ids = w.chunk_ids(0)
        n_req = [len(row) * w.chunk_tokens for row in ids]                     # what the reference arm uses
        per_step = bench.kv_bytes_of_decode(w, n_req) / w.decode_steps
        cfg = bench.workload_config(w, "all_layers", per_step)
        # the CUDA arm's figure: every visible K and V element once, summed over requests, steps and layers
        want = sum((n + w.suffix + t + 1) * w.beta for n in n_req for t in range(w.decode_steps)) * w.n_layers / w.decode_steps
        assert per_step == want and cfg["workload"] == name and cfg["layers"] == w.n_layers and cfg["decode_launch"] == "all_layers"
        assert set(cfg) == {"workload", "layers", "q_heads", "kv_heads", "head_dim", "batch", "chunks_per_request", "chunk_tokens",
                            "suffix", "decode_steps", "decode_launch", "prefill_launch", "l2", "multi_gpu"}


def test_traffic_table_names_known_workloads():
    for (name, mode), (nbytes, layers) in bench.NCU_TRAFFIC.items():
        w = mi.workload(name)
        assert mode == "all_layers" and 1 <= layers <= w.n_layers and nbytes > 0
