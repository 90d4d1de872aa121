"""The path shards by images: two CPU ranks (gloo) each run the layer table on half of a batch, and the
gathered results equal the unsharded run.  No collective sits on the data path; the gather only
brings the logits to one place for the comparison."""
from __future__ import annotations

import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import os, sys
sys.path.insert(0, os.environ["HQ_ROOT"])
import numpy as np
import torch
import torch.distributed as dist
from oracle.network import run_network
from paper_2011_10680_b200 import inputs

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
table = inputs.resnet_table(18, seed=11, image_hw=32, classes=10, width=8)
images = inputs.random_images(11, 4, 32)
per = images.shape[0] // world
mine = run_network(table, images[rank * per:(rank + 1) * per])[-1]
parts = [torch.zeros_like(torch.from_numpy(mine)) for _ in range(world)]
dist.all_gather(parts, torch.from_numpy(mine))
if rank == 0:
    whole = run_network(table, images)[-1]
    got = np.concatenate([p.numpy() for p in parts], axis=0)
    assert np.array_equal(got, whole), "sharded replicas disagree with the unsharded run"
    print("REPLICAS_OK")
dist.destroy_process_group()
'''


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_batch_sharded_replicas_match_unsharded_run(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, HQ_ROOT=ROOT, OMP_NUM_THREADS="2")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), str(script)]
    out = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "REPLICAS_OK" in out.stdout
