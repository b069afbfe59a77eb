"""The N>1 path of the benchmark (rank bookkeeping and result aggregation) on two gloo ranks."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %r)
from paper_2608_04962_b200 import dist as D
rank, local, world = D.env_world()
assert D.init("gloo")
D.barrier()
t, u = D.aggregate(10.0 + 5.0 * rank, 4096.0)
assert t == 15.0 and u == 8192.0, (t, u)
D.barrier()
D.finish()
print("ok", rank)
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_rank_aggregation_is_max_time_and_summed_units():
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD % ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT))
    for r, p in enumerate(procs):
        out = p.communicate(timeout=120)[0].decode()
        assert p.returncode == 0, out
        assert f"ok {r}" in out


def test_single_process_aggregation_is_identity():
    from paper_2608_04962_b200 import dist as D
    assert D.env_world()[2] >= 1
    assert D.aggregate(3.5, 7.0) == (3.5, 7.0)


def test_gpus_flag_against_the_launcher_environment():
    from paper_2608_04962_b200 import dist as D
    assert D.launch_plan(1, env={}) == ("run", None)
    assert D.launch_plan(4, env={}) == ("spawn", None)                     # no launcher: bench.py starts the ranks
    assert D.launch_plan(4, env={"WORLD_SIZE": "4"}) == ("run", None)
    kind, msg = D.launch_plan(8, env={"WORLD_SIZE": "2"})
    assert kind == "refuse" and "WORLD_SIZE=2" in msg
    assert D.launch_plan(1, env={"WORLD_SIZE": "2"})[0] == "refuse"
