"""The N > 1 path is "replicas only": what crosses ranks is the benchmark's aggregation (slowest
rank's time, total committed tokens).  Two gloo ranks on CPU run it."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RANK_SCRIPT = r"""
import os, sys
sys.path.insert(0, os.environ["S2D2_ROOT"])
import torch.distributed as dist
from paper_2603_25702_b200.replicas import aggregate_over_ranks, rank_prompt_seed
from s2d2_inputs import generate_prompts, get_config
rank = int(os.environ["RANK"])
assert aggregate_over_ranks(1.0, 2.0, 3, device="cpu") == (1.0, 2.0, 3)      # no group yet: identity
dist.init_process_group("gloo", rank=rank, world_size=int(os.environ["WORLD_SIZE"]))
dev_ms, wall, committed = aggregate_over_ranks(10.0 + 5.0 * rank, 0.5 - 0.1 * rank, 100 + rank, device="cpu")
assert (dev_ms, wall, committed) == (15.0, 0.5, 201), (dev_ms, wall, committed)
wl = get_config("t_bf16")
mine = generate_prompts(wl, seed=rank_prompt_seed(wl.prompt_seed, rank))
other = generate_prompts(wl, seed=rank_prompt_seed(wl.prompt_seed, 1 - rank))
assert any(len(a) != len(b) or (a != b).any() for a, b in zip(mine, other))      # replicas decode different prompts
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_two_gloo_ranks_aggregate_like_the_bench():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), S2D2_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", RANK_SCRIPT], env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out
