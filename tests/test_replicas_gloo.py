"""The N > 1 path of the benchmark on CPU: two gloo ranks, replicas only (no data-path collective);
the whole-job rate is all ranks' units over the slowest rank's time."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    from paper_2608_11688_b200 import replicas
    rank, world = replicas.init("gloo")
    assert world == 2
    replicas.barrier()
    seconds = 2.0 if rank == 0 else 4.0            # rank 1 is the slow one
    rate = replicas.whole_job_rate(48, seconds, world)
    mx = replicas.max_over_ranks(seconds)
    replicas.finish()
    print("RESULT", rank, rate, mx, flush=True)
""") % ROOT


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_gloo_ranks_report_max_time_and_whole_job_rate(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), LOCAL_RANK=str(r))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-2000:]
    for r, (o, e) in enumerate(outs):
        line = [ln for ln in o.splitlines() if ln.startswith("RESULT")][0].split()
        assert int(line[1]) == r
        assert abs(float(line[2]) - 2 * 48 / 4.0) < 1e-9       # 96 units over the slowest rank's 4 s
        assert abs(float(line[3]) - 4.0) < 1e-9


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2608_11688_b200 import replicas
    env_backup = {k: os.environ.pop(k, None) for k in ("RANK", "WORLD_SIZE")}
    try:
        assert replicas.init("gloo") == (0, 1)
        assert replicas.whole_job_rate(10, 2.0, 1) == 5.0
    finally:
        for k, v in env_backup.items():
            if v is not None:
                os.environ[k] = v
