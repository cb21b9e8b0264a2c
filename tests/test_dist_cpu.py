"""Host logic of the multi-rank benchmark, on CPU with gloo and two ranks: every rank works on its
own batch (no data-path collective) and the reported time is the maximum over ranks."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    from paper_1905_05686_b200 import synth
    dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
    rank = dist.get_rank()
    ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    worst = bench.reduce_max(ms, dist)
    layer = synth.CONFIGS["lenet_fc1"]
    mine = synth.Layer(**{**layer.__dict__, "seed": bench.rank_seed(layer.seed, rank)})
    x = synth.make_activations(mine, 4)
    w = synth.make_weights(layer)               # the layer itself is the same on every rank
    print(json.dumps({"rank": rank, "worst": worst, "x0": int(x[0, 0]), "w0": int(w[0, 0])}))
    dist.destroy_process_group()
""") % ROOT


def test_two_ranks_time_is_max_and_batches_differ(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = 29500 + os.getpid() % 2000
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, _ = p.communicate(timeout=240)
        assert p.returncode == 0
        outs.append(eval(out.strip().splitlines()[-1].replace("true", "True")))
    assert all(o["worst"] == 15.0 for o in outs)
    assert outs[0]["w0"] == outs[1]["w0"] and outs[0]["x0"] != outs[1]["x0"]


def test_single_process_reduce_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max(3.5, None) == 3.5
    assert bench.algorithmic_bytes(bench.synth.CONFIGS["alexnet_fc"], 16) == 76513280
    assert bench.dense_flops(bench.synth.CONFIGS["ffn_16384x4096"], 4096) == 2 * 4096 * 16384 * 4096
