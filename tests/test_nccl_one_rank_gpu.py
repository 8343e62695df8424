"""The collectives of multi.py on the NCCL backend, in a process group of ONE rank (the only size one GPU
allows): the barrier, the max-reduction of the elapsed time and the all-gather of a step's (out, lse) parts
run through NCCL on device tensors, and a row-range step built on them matches the plain fold step.
Runs in a child process so that the process group never meets the other tests."""
import os
import socket
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

CHILD = r"""
import os, torch, torch.distributed as dist
from paper_2605_12471_b200 import binding, multi, workloads
torch.cuda.set_device(0)
dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
dist.barrier()
assert multi.max_over_ranks(12.5, device="cuda", always=True) == 12.5
w = workloads.Workload("nccl_probe", 32, 8, 128, "bf16", 256, 1024, 500000.0)
plain = binding.cache_for(w, capacity=1024, max_chunk=256)
split = binding.cache_for(w, capacity=1024, max_chunk=256)
pos = 0
for t, n in enumerate([256, 100, 1, 33]):
    q, k, v = workloads.chunk_inputs(w, 51, t, device="cuda", n_tokens=n)
    lse = torch.empty((n, w.n_q_heads), dtype=torch.float32, device="cuda")
    want = plain.fold_step(q, k, v, lse=lse)
    got_lse = torch.empty_like(lse)
    out = split.fold_step(q, k, v, pos0=pos, lse=got_lse)
    outs, lses = multi.gather_partials(out, got_lse, always=True)        # NCCL all-gather, one rank
    assert outs.shape == (1,) + tuple(out.shape) and lses.shape == (1,) + tuple(lse.shape)
    merged, merged_lse = binding.merge_partials(outs, lses)
    torch.cuda.synchronize()
    assert torch.equal(merged.view(torch.int16), want.view(torch.int16)), t     # one part: the merge is the identity
    assert torch.allclose(merged_lse, lse, atol=1e-6), t
    pos += n
# the same step through the helper the benchmark uses
q, k, v = workloads.chunk_inputs(w, 51, 9, device="cuda", n_tokens=7)
a, _ = multi.row_range_fold_step(split, q, k, v, 0, pos, 0, 1)
b = plain.fold_step(q, k, v)
torch.cuda.synchronize()
assert torch.equal(a.view(torch.int16), b.view(torch.int16))
dist.barrier()
dist.destroy_process_group()
print("NCCL_ONE_RANK_OK")
"""


def test_collectives_of_the_benchmark_run_on_nccl_with_one_rank():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK="0", WORLD_SIZE="1", LOCAL_RANK="0",
               NCCL_NVLS_ENABLE="0")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", CHILD], cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "NCCL_ONE_RANK_OK" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
