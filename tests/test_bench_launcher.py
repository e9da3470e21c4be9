"""`bench.py --gpus N` without a launcher around it starts the N ranks itself.  The
launcher logic is checked here on CPU with a stub worker that records the rank
environment it was given."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402

STUB = textwrap.dedent("""
    import json, os, sys, time
    out, fail_rank = sys.argv[1], int(sys.argv[2])
    keys = ["RANK", "LOCAL_RANK", "WORLD_SIZE", "LOCAL_WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"]
    rank = int(os.environ["RANK"])
    with open(os.path.join(out, f"rank{rank}.json"), "w") as f:
        json.dump({k: os.environ.get(k) for k in keys}, f)
    if rank == fail_rank:
        sys.exit(7)
    if fail_rank >= 0:
        time.sleep(60)          # a healthy rank that would wait for the failed one
""")


def _stub(tmp_path):
    path = os.path.join(tmp_path, "stub_worker.py")
    with open(path, "w") as f:
        f.write(STUB)
    return path


def test_spawn_ranks_gives_every_rank_its_environment(tmp_path):
    world = 3
    codes = bench.spawn_ranks(world, [sys.executable, _stub(tmp_path), str(tmp_path), "-1"])
    assert codes == [0] * world
    envs = [json.load(open(os.path.join(tmp_path, f"rank{r}.json"))) for r in range(world)]
    for r, e in enumerate(envs):
        assert e["RANK"] == str(r) and e["LOCAL_RANK"] == str(r)
        assert e["WORLD_SIZE"] == str(world) and e["LOCAL_WORLD_SIZE"] == str(world)
        assert e["MASTER_ADDR"] == "127.0.0.1"
    assert len({e["MASTER_PORT"] for e in envs}) == 1 and int(envs[0]["MASTER_PORT"]) > 0


def test_spawn_ranks_stops_the_others_when_one_rank_fails(tmp_path):
    import time
    t0 = time.time()
    codes = bench.spawn_ranks(2, [sys.executable, _stub(tmp_path), str(tmp_path), "1"])
    assert codes[1] == 7 and codes[0] not in (0, None)        # rank 0 was terminated, not left waiting
    assert time.time() - t0 < 30


def test_rank_environment_does_not_leak_into_the_parent():
    before = dict(os.environ)
    env = bench.rank_environment(1, 4, 29999)
    assert env["RANK"] == "1" and env["WORLD_SIZE"] == "4" and env["MASTER_PORT"] == "29999"
    assert dict(os.environ) == before


def _bench(args, env=None):
    e = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    e.update(env or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, cwd=ROOT, env=e,
                          capture_output=True, text=True, timeout=600)


def test_gpus_flag_is_never_silently_ignored():
    # more GPUs asked for than the machine shows: refuse, do not time one GPU and call it N
    import torch
    want = torch.cuda.device_count() + 1 if torch.cuda.is_available() else 2
    out = _bench(["--gpus", str(max(want, 2)), "--steps", "1"])
    assert out.returncode != 0 and "CUDA device" in out.stderr and out.stdout.strip() == ""
    # a launcher's world size that contradicts --gpus
    out = _bench(["--gpus", "2", "--steps", "1"], {"WORLD_SIZE": "3", "RANK": "0", "LOCAL_RANK": "0"})
    assert out.returncode != 0 and "contradicts" in out.stderr and out.stdout.strip() == ""
