"""The process-group code paths of ps.py and sharded.py on the GPU with NCCL.  Only one GPU is
available, so the group has a single rank: the collectives (all-to-all, all-gather, all-reduce)
really run through NCCL on device tensors, but move nothing between devices.  The multi-rank
logic of the same functions is covered by the gloo tests on CPU and by the emulated ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist

from paper_1905_10936_b200 import ps
from paper_1905_10936_b200 import workloads as wl
from paper_1905_10936_b200.engine import EFEngine
from paper_1905_10936_b200.sharded import DistributedShard

pytestmark = pytest.mark.gpu

TILE = 4096


@pytest.fixture(scope="module")
def nccl_world1():
    if not dist.is_nccl_available():
        pytest.skip("NCCL is not available in this torch build")
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        yield
    finally:
        torch.cuda.synchronize()
        dist.destroy_process_group()


def test_parameter_server_step_through_nccl(nccl_world1):
    sizes = [3 * TILE + 5, 640, 10, 4 * TILE]
    w = wl.custom_workload("ps-nccl", sizes, 1, steps=3, scale_range=(1e-2, 1.0), config_id=700)
    ref = EFEngine(w.offsets, 1, w.mu, w.eta)
    rk = ps.Rank(EFEngine(w.offsets, 1, w.mu, w.eta, one_local_worker=True), w.sizes, 0, 1)
    es = w.element_scales("cuda")
    for t in range(w.steps):
        g = w.draw_grad(t, 0, "cuda", es)
        ref.worker_step(0, g)
        ref.server_step()
        ps.step(rk, g)                       # all_to_all_single and all_gather_into_tensor on CUDA tensors
        assert torch.equal(rk.engine.params(), ref.params())
        assert torch.equal(rk.engine.residual(-1), ref.residual(-1))
    sc, wd = ps.unpack_message(rk.update.cpu().numpy(), w.sizes, 0, w.B)
    assert np.array_equal(sc, ref.server_scales().cpu().numpy())
    assert np.array_equal(wd, ref.server_words().cpu().numpy().view(np.uint32))


def test_distributed_shard_through_nccl(nccl_world1):
    sizes = [5 * TILE, 777, 2 * TILE + 36]
    w = wl.custom_workload("shard-nccl", sizes, 3, steps=3, scale_range=(1e-2, 1.0), config_id=701)
    ref = EFEngine(w.offsets, w.M, w.mu, w.eta)
    ds = DistributedShard(w.sizes, w.M, w.mu, w.eta, 0, 1)
    assert not ds.any_cut and (ds.shard.elem_lo, ds.shard.elem_hi) == (0, w.d)
    es = w.element_scales("cuda")
    stride = (w.d + 3) // 4 * 4
    gall = torch.zeros(w.M, stride, device="cuda")
    for t in range(w.steps):
        for i in range(w.M):
            w.draw_grad(t, i, "cuda", es, out=gall[i, :w.d])
        ref.worker_step_all(gall); ref.server_step()
        ds.worker_step_all(gall); ds.server_step()
        assert torch.equal(ds.eng.params(), ref.params())
    # force the exchange path although nothing is cut: the all-reduce of B zeros must be harmless
    ds.any_cut = True
    for i in range(w.M):
        w.draw_grad(9, i, "cuda", es, out=gall[i, :w.d])
    ref.worker_step_all(gall); ref.server_step()
    ds.worker_step_all(gall); ds.server_step()
    assert torch.equal(ds.eng.params(), ref.params())


def test_push_variant_over_symmetric_memory(nccl_world1):
    """The push variant as a multi-device run sets it up: buffers in symmetric memory, peer
    addresses from the rendezvous, barriers as all-reduces.  With one rank the only peer is the
    rank itself."""
    try:
        import torch.distributed._symmetric_memory  # noqa: F401
    except ImportError:
        pytest.skip("this torch build has no symmetric memory")
    sizes = [3 * TILE + 5, 640, 10, 4 * TILE]
    w = wl.custom_workload("ps-symm", sizes, 1, steps=3, scale_range=(1e-2, 1.0), config_id=702)
    ref = EFEngine(w.offsets, 1, w.mu, w.eta)
    recv, update, recv_ptrs, update_ptrs = ps.symmetric_buffers(w.sizes, 0, 1, torch.device("cuda", 0))
    rk = ps.Rank(EFEngine(w.offsets, 1, w.mu, w.eta, one_local_worker=True), w.sizes, 0, 1,
                 recv=recv, update=update)
    rk.connect(recv_ptrs, update_ptrs)
    flag = torch.zeros(1, device="cuda")
    es = w.element_scales("cuda")
    for t in range(w.steps):
        g = w.draw_grad(t, 0, "cuda", es)
        ref.worker_step(0, g)
        ref.server_step()
        ps.step_push(rk, g, flag)
        assert torch.equal(rk.engine.params(), ref.params())
        assert torch.equal(rk.engine.residual(-1), ref.residual(-1))
    sc, wd = ps.unpack_message(rk.update.cpu().numpy(), w.sizes, 0, w.B)
    assert np.array_equal(sc, ref.server_scales().cpu().numpy())
    assert np.array_equal(wd, ref.server_words().cpu().numpy().view(np.uint32))


@pytest.mark.parametrize("push", [False, True])
def test_bench_process_group_mode_runs_with_one_rank(push):
    """bench.py --workload ps --process-group: the mode torchrun uses with one rank per GPU."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    cmd = [sys.executable, os.path.join(root, "bench.py"), "--workload", "ps", "--process-group", "--config", "1",
           "--steps", "3", "--warmup", "3"] + (["--push"] if push else [])
    out = subprocess.run(cmd, capture_output=True, text=True, env=env, cwd=root, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([ln for ln in out.stdout.splitlines() if ln.startswith("{")][-1])
    assert line["run"]["variant"] == ("push" if push else "collective") and line["run"]["process_group"] == "nccl"
    assert line["value"] > 0 and line["gpu_launches"] > 0
