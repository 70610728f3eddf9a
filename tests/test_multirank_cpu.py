"""Host-side logic of the multi-rank paths, run as 2 gloo ranks on CPU (no GPU needed).

1. Row-sharded quantization protocol: every rank reduces its own rows (Eq. 1 numerator), the ranks
   exchange one float with all-reduce(max), each rank encodes its rows with the shared alpha.  The
   concatenation must equal the single-process result bit for bit.  On a GPU machine the per-rank
   compute calls are abs_amax / abs_quantize_ex(ABS_F_ALPHA_GIVEN); here the CPU oracle stands in
   for them so that the protocol itself (sharding, the 4-byte exchange, reassembly) is what is tested.
2. bench.py's reference arm under a 2-rank launch: rank 0 alone prints one JSON line, rank 1 exits 0.
"""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _shard_worker(rank, world, port, out_dir):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    from oracle import abs_oracle as O
    from paper_2603_28765_b200 import inputs as I
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    xb = I.generate("cfg2", 96, 512)
    rows = xb.shape[0]
    lo, hi = rows * rank // world, rows * (rank + 1) // world
    local = np.ascontiguousarray(xb[lo:hi])
    a = torch.tensor([float(O.amax(local))], dtype=torch.float32)
    dist.all_reduce(a, op=dist.ReduceOp.MAX)                       # the only exchange: 4 bytes
    alpha = O.alpha_from_amax(O.FMT_IF4, np.float32(a.item()))
    c, s, _ = O.quantize(O.FMT_IF4, local, flags=O.F_ALPHA_GIVEN, alpha=alpha)
    # the same shard with stochastic rounding: App. B's stream runs over the whole tensor, so the shard passes the
    # index of its first element
    cs, ss, _ = O.quantize(O.FMT_IF4, local, flags=O.F_ALPHA_GIVEN | O.F_STOCHASTIC, alpha=alpha, sr_seed=31,
                           sr_index_offset=lo * xb.shape[1])
    np.save(os.path.join(out_dir, f"sr_codes{rank}.npy"), cs)
    np.save(os.path.join(out_dir, f"sr_scales{rank}.npy"), ss)
    np.save(os.path.join(out_dir, f"codes{rank}.npy"), c)
    np.save(os.path.join(out_dir, f"scales{rank}.npy"), s)
    np.save(os.path.join(out_dir, f"alpha{rank}.npy"), np.array([alpha], np.float32))
    dist.barrier()
    dist.destroy_process_group()


def test_row_sharded_protocol_matches_single_process(tmp_path):
    import torch.multiprocessing as mp
    from oracle import abs_oracle as O
    from paper_2603_28765_b200 import inputs as I
    world, port = 2, _free_port()
    mp.spawn(_shard_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    xb = I.generate("cfg2", 96, 512)
    c, s, a = O.quantize(O.FMT_IF4, xb)
    codes = np.concatenate([np.load(tmp_path / f"codes{r}.npy") for r in range(world)])
    scales = np.concatenate([np.load(tmp_path / f"scales{r}.npy") for r in range(world)])
    assert np.array_equal(codes, c) and np.array_equal(scales, s)
    for r in range(world):
        assert np.load(tmp_path / f"alpha{r}.npy")[0] == a
    cs, ss, _ = O.quantize(O.FMT_IF4, xb, flags=O.F_STOCHASTIC, sr_seed=31)
    assert np.array_equal(np.concatenate([np.load(tmp_path / f"sr_codes{r}.npy") for r in range(world)]), cs)
    assert np.array_equal(np.concatenate([np.load(tmp_path / f"sr_scales{r}.npy") for r in range(world)]), ss)


def test_reference_arm_prints_once_under_two_ranks():
    port = _free_port()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "1", "--warmup", "0"]
    env = dict(os.environ, OMP_NUM_THREADS="1")
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["unit"] == "GB/s"
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["e2e"]["h2d_bytes_per_step"] == 0
    assert rec["value"] > 0
