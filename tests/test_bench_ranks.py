"""The one-process-per-GPU plumbing of bench.py on CPU: two gloo ranks, and the reference arm under torchrun."""
import json
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(nproc, script_args, env_extra=None, timeout=600):
    env = dict(os.environ)
    env.update(env_extra or {})
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(nproc),
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port())] + script_args
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_max_over_ranks_and_sharded_seeds_with_two_gloo_ranks(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(textwrap.dedent("""
        import json, os, sys
        sys.path.insert(0, %r)
        import bench
        rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
        r = bench.Ranks(world, backend="gloo")
        r.barrier()
        slowest = r.max(1.0 + rank)                       # every rank must learn the slowest rank's time
        cfg = bench.workload_config("8b_b1", rank)        # each rank verifies its own batch of the same model
        rec = {"rank": rank, "max": slowest, "seed": cfg.seed, "weight_seed": cfg.weight_seed,
               "value": bench.aggregate(world, 8, slowest)}
        os.write(1, (json.dumps(rec) + chr(10)).encode())   # one write per line: the ranks share the pipe
        r.close()
    """ % ROOT))
    out = _torchrun(2, [str(script)])
    assert out.returncode == 0, out.stderr[-2000:]
    recs = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert sorted(r["rank"] for r in recs) == [0, 1]
    assert all(r["max"] == 2.0 for r in recs)
    assert len({r["seed"] for r in recs}) == 2 and len({r["weight_seed"] for r in recs}) == 1
    assert all(abs(r["value"] - 2 * 8 / 2.0e-3) < 1e-9 for r in recs)   # job-wide units / slowest step


def test_reference_arm_prints_one_line_from_rank_zero_only():
    out = _torchrun(2, ["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                        "--workload", "tiny", "--oracle-rows", "10"])
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["gpu_launches"] == 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["cpu_baseline"]["value"] == rec["value"]
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["e2e"]["value"] == rec["value"]
    assert rec["config"]["workload"] == "tiny" and rec["vs_baseline"] is None


def test_vocabulary_shard_bounds_cover_the_vocabulary_once():
    import bench
    for V, G in ((128256, 1), (128256, 2), (128256, 8), (152064, 4), (4099, 3), (100, 8)):
        b = bench.shard_bounds(V, G)
        assert len(b) == G and b[0][0] == 0 and b[-1][1] == V
        assert all(lo <= hi for lo, hi in b) and all(b[i][1] == b[i + 1][0] for i in range(G - 1))
        assert all(lo % 16 == 0 for lo, hi in b if hi > lo)          # non-empty slices start on a 16-row boundary


def test_row_partials_are_gathered_rank_major_with_two_gloo_ranks(tmp_path):
    script = tmp_path / "gather.py"
    script.write_text(textwrap.dedent("""
        import json, os, sys
        sys.path.insert(0, %r)
        import torch, bench
        rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
        r = bench.Ranks(world, backend="gloo")
        R = 5
        part = torch.full((R, 4), float(rank)) + torch.arange(R).float()[:, None] * 10     # [R, 4] per rank
        gathered = torch.empty((world, R, 4))
        r.all_gather(gathered, part)                           # the layout wisv_verify_gathered expects: [G][R]
        ok = all(bool((gathered[g] == torch.full((R, 4), float(g)) + torch.arange(R).float()[:, None] * 10).all())
                 for g in range(world))
        rec = {"rank": rank, "ok": ok, "shape": list(gathered.shape)}
        os.write(1, (json.dumps(rec) + chr(10)).encode())   # one write per line: the ranks share the pipe
        r.close()
    """ % ROOT))
    out = _torchrun(2, [str(script)])
    assert out.returncode == 0, out.stderr[-2000:]
    recs = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(recs) == 2 and all(r["ok"] and r["shape"] == [2, 5, 4] for r in recs)


def test_model_weights_are_generated_once_and_shared_between_two_gloo_ranks(tmp_path):
    """With several ranks rank 0 draws the LM head once and the others map its file; all ranks end up with the same
    model, the batches still differ, and the file is gone after the job."""
    script = tmp_path / "weights.py"
    script.write_text(textwrap.dedent("""
        import hashlib, json, os, sys
        sys.path.insert(0, %r)
        import numpy as np
        import bench, gen
        bench.SHM_DIR = %r
        rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
        r = bench.Ranks(world, backend="gloo")
        cfg = gen.config("tiny").with_(weight_seed=77, seed=5 + 1000 * rank)     # one model, a batch per rank
        w, path = bench.shared_weights(cfg, rank, r)
        same = all(np.array_equal(np.asarray(w[k]), gen.make_weights(cfg)[k]) for k in ("lm_head", "W1", "b1", "w2"))
        rec = {"rank": rank, "same": bool(same), "owner": path is not None,
               "mapped": isinstance(w["lm_head"], np.memmap), "files": sorted(os.listdir(%r))}
        r.barrier()
        if path:
            os.unlink(path)
        os.write(1, (json.dumps(rec) + chr(10)).encode())
        r.close()
    """ % (ROOT, str(tmp_path / "shm"), str(tmp_path / "shm"))))
    (tmp_path / "shm").mkdir()
    out = _torchrun(2, [str(script)])
    assert out.returncode == 0, out.stderr[-2000:]
    recs = sorted((json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")), key=lambda r: r["rank"])
    assert [r["rank"] for r in recs] == [0, 1] and all(r["same"] for r in recs)
    assert recs[0]["owner"] and not recs[1]["owner"] and recs[1]["mapped"] and not recs[0]["mapped"]
    assert all(len(r["files"]) == 1 and r["files"][0].endswith(".npy") for r in recs)
    assert os.listdir(tmp_path / "shm") == []
