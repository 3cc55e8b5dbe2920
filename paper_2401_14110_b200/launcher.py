"""Start one process per GPU on this node (the data-parallel split of App. C.1: every rank its own rows).

``bench.py --gpus N`` calls this when no launcher environment (WORLD_SIZE) is present, so that N always means N
ranks.  The ranks are started through ``torch.distributed.run`` with a rendezvous on 127.0.0.1; each child sees
RANK, LOCAL_RANK and WORLD_SIZE exactly as under an external launcher.
"""
import socket
import subprocess
import sys


def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_command(n_ranks: int, argv, port: int):
    """The command line that starts ``n_ranks`` copies of ``argv`` (a script path followed by its arguments)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
            "--master-addr", "127.0.0.1", "--master-port", str(port)] + list(argv)


def spawn_ranks(n_ranks: int, argv, devices=None, env=None) -> int:
    """Run ``argv`` as ``n_ranks`` ranks and return the launcher's exit code.

    ``devices`` is the number of GPUs visible to this process; asking for more ranks than devices is refused
    (exit code 2 and a message on stderr) rather than run with fewer ranks than requested."""
    if n_ranks < 1:
        raise ValueError("n_ranks must be positive")
    if devices is not None and devices < n_ranks:
        sys.stderr.write(f"--gpus {n_ranks}: only {devices} GPU(s) are visible to this process; refusing to run fewer "
                         "ranks than requested\n")
        return 2
    return subprocess.run(launch_command(n_ranks, argv, free_port()), env=env).returncode
