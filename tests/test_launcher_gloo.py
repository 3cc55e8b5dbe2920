"""`bench.py --gpus N` must mean N ranks.  The launcher that starts them is exercised here with two gloo ranks on
CPU: two processes come up, see RANK / LOCAL_RANK / WORLD_SIZE, and meet in a collective; asking for more ranks than
devices is refused instead of quietly running fewer."""
import os
import sys

from paper_2401_14110_b200 import launcher

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HELPER = os.path.join(ROOT, "tests", "helpers", "rank_report.py")


def test_two_ranks_are_started_and_meet(tmp_path):
    rc = launcher.spawn_ranks(2, [HELPER, str(tmp_path)])
    assert rc == 0
    seen = sorted(os.listdir(tmp_path))
    assert seen == ["rank0.txt", "rank1.txt"]
    rows = [open(os.path.join(tmp_path, n)).read().split() for n in seen]
    assert [r[0] for r in rows] == ["0", "1"] and all(r[1] == "2" for r in rows)
    assert [r[2] for r in rows] == ["0", "1"]                 # one local rank per process
    assert all(r[3] == "3" for r in rows)                     # both took part in the all-reduce: 1 + 2
    assert rows[0][4] != rows[1][4]                           # two processes


def test_more_ranks_than_devices_is_refused(capsys):
    assert launcher.spawn_ranks(8, [HELPER, "/nonexistent"], devices=1) == 2
    assert "refusing" in capsys.readouterr().err


def test_launch_command_uses_the_loopback_rendezvous():
    cmd = launcher.launch_command(4, ["bench.py", "--gpus", "4"], 29999)
    assert cmd[0] == sys.executable and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-3:] == ["bench.py", "--gpus", "4"]
