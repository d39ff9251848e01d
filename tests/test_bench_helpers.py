"""Host-side helpers of bench.py (no GPU): the generation-index spread, the oracle sample
size shared by both arms, and the command that starts the replica processes for --gpus N."""
import importlib.util
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_generation_indices_cover_the_run():
    b = _bench()
    full = b.gen_indices(255)
    assert full == list(range(1, 256))                       # K = 255 is the run itself
    few = b.gen_indices(20)
    assert few[0] == 1 and few[-1] <= 255 and few == sorted(few) and len(set(few)) == 20
    assert few[-1] > 230                                      # spread over the whole run, not its start
    many = b.gen_indices(300)
    assert len(many) == 300 and min(many) == 1 and max(many) == 255


def test_oracle_sample_is_the_same_rule_in_both_arms():
    b = _bench()
    assert b.oracle_steps(20) == 20 and b.oracle_steps(5) == 8 and b.oracle_steps(255) == b.ORACLE_STEPS


def test_replica_processes_are_started_with_the_standard_launcher(monkeypatch):
    b = _bench()
    seen = {}

    def fake_call(cmd):
        seen["cmd"] = cmd
        return 0
    monkeypatch.setattr(b.subprocess, "call", fake_call)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "7", "--warmup", "3"])

    class Args:
        gpus = 4
    assert b.spawn_replicas(Args) == 0
    cmd = seen["cmd"]
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert int(cmd[cmd.index("--master-port") + 1]) > 0
    assert cmd[-6:] == ["--gpus", "4", "--steps", "7", "--warmup", "3"]
    assert os.path.basename(cmd[-7]) == "bench.py"
