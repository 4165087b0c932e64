"""Host-side logic of the N>1 bench path, run as two gloo ranks on the CPU: every rank is an
independent replica, the slowest rank sets the time, the value is the sum of all replicas'
work over that time, and only rank 0 reports."""
import os
import socket
import subprocess
import sys
import json

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    step = [0.5, 0.8][rank]                 # rank 1 is slower
    kern = [0.45, 0.4][rank]
    got = bench.max_over_ranks(dist, [step, kern])
    value = bench.replica_throughput(world, 4.0e9, got[0])
    out.put((rank, got, value))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_take_the_slowest_time_and_sum_the_work():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, value in res:
        assert got == [0.8, 0.45]
        assert value == 2 * 4.0e9 / 0.8


def test_single_rank_passthrough():
    import bench
    assert bench.max_over_ranks(None, [1.0, 2.0]) == [1.0, 2.0]
    assert bench.replica_throughput(1, 10.0, 2.0) == 5.0


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "1",
                        "--shrink", "6", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env.update(RANK="0", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "1",
                        "--shrink", "6", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0


def test_direction_aware_roofline_and_config_record():
    """Host logic of the benchmark line: the floor of a launch is the slower direction of the link,
    both arms describe the configuration with the same keys, and every ncu figure the line quotes
    names a summary that is in the tree."""
    import os
    import bench
    link = {"ce_h2d_gbs": 50.0, "ce_d2h_gbs": 60.0, "sm_h2d_gbs": 48.0, "sm_d2h_gbs": 52.0}
    r = bench.link_roofline(8e9, 4e9, 0.2, link)                  # 8 GB in, 4 GB out in 200 ms
    assert r["direction"] == "host_to_device" and abs(r["floor_ms"] - 160.0) < 1e-9
    assert abs(r["frac"] - 0.8) < 1e-12 and abs(r["achieved"] - 40.0) < 1e-9 and r["peak"] == 50.0
    r = bench.link_roofline(1e9, 6e9, 0.2, link)
    assert r["direction"] == "device_to_host" and abs(r["frac"] - 0.5) < 1e-12
    a, b = bench.config_of(5, 0), bench.config_of(5, 0)
    assert a == b and a["cfg"] == 5 and a["pool_bytes"] == 16 << 30 and a["page_bytes"] == 2 << 20
    assert bench.config_of(3, 0)["frames"] == 9216
    root = os.path.dirname(os.path.abspath(bench.__file__))
    for cfg, (nbytes, name, sectors, how) in bench.NCU_LINK_TRAFFIC.items():
        text = open(os.path.join(root, "profiles", name)).read().replace(" ", "").replace(",", "")
        assert str(sectors) in text, (cfg, name)                  # the sector count is in the committed summary
        assert nbytes >= sectors * 32
