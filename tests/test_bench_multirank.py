"""The N > 1 path of bench.py on CPU: two gloo ranks.  The path has no exchange step (replicas only), so what the
ranks share is the timing rule: barrier, maximum of the per-rank times, whole-job throughput = N * T / max time."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch
    import bench
    rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
    torch.distributed.init_process_group("gloo")
    torch.distributed.barrier()
    mine = [0.004 + 0.001 * rank, 0.010 - 0.002 * rank]          # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(mine, "cpu")
    torch.distributed.barrier()
    if rank == 0:
        print(json.dumps({"got": got, "value": bench.whole_job_value(64, world, got[0])}))
    torch.distributed.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_take_the_maximum_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29613", str(script)],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert abs(res["got"][0] - 0.005) < 1e-12 and abs(res["got"][1] - 0.010) < 1e-12
    assert abs(res["value"] - 2 * 64 / 0.005) < 1e-6


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], "cpu") == [1.5, 2.5]
    assert bench.whole_job_value(64, 1, 0.004) == 16000.0


def test_byte_model_matches_the_papers_bytes_per_token():
    """The per-layer weight bytes reproduce the paper's streamed bytes per token for the non-speculative baseline
    (Table 4: 12.95 GB for the 32 layers of a 7B model) and the cascaded method's figures (Eq. 4, Table 5)."""
    from paper_2605_11186_b200 import roofline, inputs as gen
    per_layer = roofline.layer_weight_bytes(gen.LLAMA_7B)
    assert per_layer == 404_750_336
    assert abs(32 * per_layer / 1e9 - 12.95) < 0.01
    # Eq. 4: gamma draft passes over 3 layers + one pass over the other 29 layers, per accepted token
    draft, rest = 3 * per_layer / 1e9, 29 * per_layer / 1e9
    assert abs((5 * draft + rest) / 3.0520 - 5.8354) < 0.01      # Table 5, gamma = 5
    assert abs((3 * draft + rest) / 2.7077 - 5.6805) < 0.01      # Table 5, gamma = 3
    # totals of the hot-path table for config 3
    assert roofline.forward_bytes(gen.LLAMA_7B, 512, 16) == 13_500_030_976
    assert roofline.forward_bytes(gen.LLAMA_7B, 512, 128) == 13_618_388_992
    assert roofline.forward_bytes(gen.LLAMA_13B, 2048, 64) == 27_487_283_200
