"""One rank of a learner-per-process job, run as a child process by test_exchange.py.

usage: exchange_worker.py <cpu|cpu-nopeer|gpu|gpu-peer|gpu-flags> <topk|chunk|layer_topk> <d> <steps>      (RANK, WORLD_SIZE, MASTER_* from the env)

Every rank generates all learners' seeded inputs, takes the learner of its own rank through
multi.LearnerRank, and checks each step's index list, reduced values, its learner's memory and
its weight replica, bit for bit, against the oracle's single-process step over all learners.

"gpu": the library's kernels on cuda:0 (the ranks share the device; nothing in a kernel waits for
another rank, the exchanges are gloo collectives between launches).
"gpu-peer": as "gpu", with the all-gather fused into the compressing kernel (stores into the other processes'
gathered-rows buffers, mapped with CUDA IPC).
"gpu-flags": as "gpu-peer" without the fence: the reducing kernel waits for flag words the compressing kernels
set.  Only for a single rank here: kernels of different processes that wait for one another must not share a device.
"cpu-nopeer": as "cpu", but the ranks ask for the fused exchange (exchange="peer") while a stand-in for the
device query reports that no rank can reach a peer's memory: every rank must fall back to the collective exchange,
with a warning, before anything is mapped or stored, and the results stay those of the single-process step.
"cpu": the same orchestration over an engine made of the oracle's pieces, so that leader rotation,
broadcast source and row order are checked where there is no GPU.
"""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2104_11125_b200 import binding, multi, workloads  # noqa: E402


class OracleEngine:
    """Test-only stand-in with the three calls LearnerRank makes, on CPU tensors."""

    def __init__(self, d, k, beta, lr, selector, layers):
        self.d, self.k, self.beta, self.lr, self.selector, self.layers = d, k, beta, lr, selector, layers

    def select(self, g, m, out_idx):
        acc = oracle.accumulate(g.numpy(), m.numpy())
        if self.selector == "layer_topk":
            idx, _ = oracle.layer_topk(acc, *self.layers)
        else:
            idx, _ = (oracle.chunk_select if self.selector == "chunk" else oracle.topk)(acc, self.k)
        out_idx.copy_(torch.from_numpy(idx))
        self.last = out_idx.clone()

    def compress(self, g, m, idx, out):
        if idx is None:                                  # the leader: the list of the select() just before
            idx, self.last = self.last, None
        sel = np.zeros(self.d, np.uint8)
        sel[idx.numpy()] = 1
        out.copy_(torch.from_numpy(oracle.learner(g.numpy(), m.numpy(), idx.numpy(), sel, self.beta)))

    def reduce_rows(self, rows, val, idx=None, weights=None):
        val.copy_(torch.from_numpy(oracle.reduce(rows.view(-1, self.k).numpy())))
        if weights is not None:
            oracle.apply(weights.numpy(), idx.numpy(), val.numpy(), self.lr)


def main():
    mode, selector, d, steps = sys.argv[1], sys.argv[2], int(sys.argv[3]), int(sys.argv[4])
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    assert not (mode == "gpu-flags" and world > 1), "ranks that wait for one another need a GPU each"
    w = workloads.TINY.scaled(d, world)
    k, beta, lr = w.k, w.beta, w.lr
    layers = None
    if selector == "layer_topk":                     # five layers of uneven size and rate, the first sent whole
        sizes = [97, d // 3, 1, d // 5, 0]
        sizes[4] = d - sum(sizes)
        keep = [97, max(1, d // 300), 1, max(1, d // 1000), 0]
        keep[4] = k - sum(keep)
        assert 1 <= keep[4] <= sizes[4]
        layers = (sizes, keep)
    exchange = {"gpu-peer": "peer", "gpu-flags": "peer-flags"}.get(mode, "collective")
    if exchange != "collective":
        mode = "gpu"
    dev = torch.device("cuda", 0) if mode == "gpu" else torch.device("cpu")
    if mode == "gpu":
        torch.cuda.set_device(dev)
        node = multi.LearnerRank(d, k, beta, lr, layers=layers, exchange=exchange,
                                 selector={"topk": binding.SELECTOR_TOPK, "chunk": binding.SELECTOR_CHUNK,
                                           "layer_topk": binding.SELECTOR_LAYER_TOPK}[selector])
    elif mode == "cpu-nopeer":
        import warnings
        asked = []

        def no_access(this_device, peer_device):
            asked.append((this_device, peer_device))
            return False

        with warnings.catch_warnings(record=True) as caught:
            warnings.simplefilter("always")
            node = multi.LearnerRank(d, k, beta, lr, engine=OracleEngine(d, k, beta, lr, selector, layers), device=dev,
                                     exchange="peer", can_access_peer=no_access)
        assert node.exchange == "collective", "the rank kept exchange=%r without peer access" % node.exchange
        assert any("falls back" in str(c.message) for c in caught), "no warning about the fallback"
        assert not hasattr(node, "peer_rows"), "buffers were mapped although a peer is out of reach"
    else:
        node = multi.LearnerRank(d, k, beta, lr, engine=OracleEngine(d, k, beta, lr, selector, layers), device=dev)
    prof = workloads.profile(w, dev)
    m_o = [x.cpu().numpy().copy() for x in workloads.initial_memory(w, dev)]
    th_o = workloads.initial_weights(w, dev).cpu().numpy().copy()
    mem = torch.from_numpy(m_o[rank].copy()).to(dev)
    theta = torch.from_numpy(th_o.copy()).to(dev)
    for t in range(steps):
        g_dev = workloads.gradients(w, t, dev, prof)
        g_all = [g.cpu().numpy() for g in g_dev]
        grad = g_dev[rank].contiguous()
        idx, val = node.step(grad, mem, theta, t)
        if mode == "gpu":
            torch.cuda.synchronize()
            assert node.engine.status() == binding.OK
        idx_o, val_o, _ = oracle.step(g_all, m_o, th_o, t, k, beta, lr, want_gathered=False,
                                      selector="topk" if selector == "layer_topk" else selector, layers=layers)
        assert np.array_equal(idx.cpu().numpy(), idx_o), "step %d rank %d: index lists differ" % (t, rank)
        assert np.array_equal(val.cpu().numpy(), val_o), "step %d rank %d: reduced values differ" % (t, rank)
        assert np.array_equal(mem.cpu().numpy(), m_o[rank]), "step %d rank %d: memory differs" % (t, rank)
        assert np.array_equal(theta.cpu().numpy(), th_o), "step %d rank %d: weights differ" % (t, rank)
    assert node.exchange_bytes() == (4 * k * world if world > 1 else 0)
    node.close()
    dist.barrier()
    dist.destroy_process_group()
    print("rank", rank, "ok")


if __name__ == "__main__":
    main()
