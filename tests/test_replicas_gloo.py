"""world_size-2 check of the multi-GPU reporting rule on CPU (gloo): time = max over
ranks, work = sum over ranks; no data-path collective exists on this path."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
from paper_2607_17181_b200.replicas import job_totals
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%s" % sys.argv[2], rank=int(sys.argv[3]), world_size=2)
rank = dist.get_rank()
ms, units = job_totals(100.0 + 50.0 * rank, 9.5e9 * (rank + 1), dist)
assert ms == 150.0, ms
assert units == 9.5e9 * 3, units
dist.barrier()
dist.destroy_process_group()
print("ok", rank)
"""


def test_two_replicas_report_max_time_and_summed_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = str(29500 + os.getpid() % 2000)
    procs = [subprocess.Popen([sys.executable, str(script), ROOT, port, str(r)], stdout=subprocess.PIPE,
                              stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert all("ok" in o for o in outs)


def test_single_replica_is_identity():
    from paper_2607_17181_b200.replicas import job_totals
    assert job_totals(12.5, 3.0) == (12.5, 3.0)
