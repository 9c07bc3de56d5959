"""Worker for the world_size-2 gloo test of the coordinate-sharded step's orchestration.

Each rank holds a stand-in shard that follows the phase protocol of include/efcp.h
(efcp_shard_phase / efcp_shard_buffer) on CPU tensors in plain numpy, so that
paper_2306_06098_b200.sharded.ShardedStep and its all-reduce exchanges can run without a
GPU.  Rank 0 gathers the pieces and compares them with the unsharded CPU oracle.
Launched by tests/test_multiprocess.py through torch.distributed.run."""
import json
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

BITS = (12, 10, 9)  # digits of the 31-bit magnitude key, most significant first


def pick(hist, k_rem):
    """Bin b with count(bins > b) < k_rem <= count(bins >= b), and k_rem - count(bins > b)."""
    above = 0
    for b in range(len(hist) - 1, -1, -1):
        if above < k_rem <= above + int(hist[b]):
            return b, k_rem - above
        above += int(hist[b])
    raise AssertionError("histogram short of k")


class NumpyShard:
    def __init__(self, d_lo, d_hi, m, k_global, lam, index, count):
        self.lo, self.hi, self.m, self.k, self.lam = d_lo, d_hi, m, k_global, np.float32(lam)
        self.index, self.count = index, count
        n = d_hi - d_lo
        self.e = np.zeros(n, np.float32)
        self.rows = [(np.zeros(0, np.int64), np.zeros(0, np.float32)) for _ in range(m)]
        self.S = np.zeros((m, m))
        self.t = 0
        self.calls = []
        self.buf = [torch.zeros(1 << BITS[0], dtype=torch.int32),
                    torch.zeros(1 << BITS[1], dtype=torch.int32),
                    torch.zeros(1 << BITS[2], dtype=torch.int32),
                    torch.zeros(2 * count, dtype=torch.int32),
                    torch.zeros(m, dtype=torch.float64)]

    def shard_buffer(self, phase):
        return self.buf[phase]

    def shard_phase(self, phase, grad=None, update=None, stream=None):
        self.calls.append((phase, grad is not None, update is not None))
        if phase == 0:
            self.a = self.e + grad.numpy()
            self.key = self.a.view(np.uint32) & np.uint32(0x7FFFFFFF)
            self.buf[0][:] = torch.from_numpy(np.bincount(self.key >> 19, minlength=4096).astype(np.int32))
        elif phase == 1:
            self.b1, self.k1 = pick(self.buf[0].numpy(), self.k)
            sel = self.key[(self.key >> 19) == self.b1]
            self.buf[1][:] = torch.from_numpy(np.bincount((sel >> 9) & 1023, minlength=1024).astype(np.int32))
        elif phase == 2:
            self.b2, self.k2 = pick(self.buf[1].numpy(), self.k1)
            sel = self.key[(self.key >> 9) == ((self.b1 << 10) | self.b2)]
            self.buf[2][:] = torch.from_numpy(np.bincount(sel & 511, minlength=512).astype(np.int32))
        elif phase == 3:
            b3, self.n_eq = pick(self.buf[2].numpy(), self.k2)
            self.T = (self.b1 << 19) | (self.b2 << 9) | b3
            self.buf[3].zero_()
            self.buf[3][2 * self.index] = int((self.key > self.T).sum())
            self.buf[3][2 * self.index + 1] = int((self.key == self.T).sum())
        elif phase == 4:
            tot = self.buf[3].numpy().astype(np.int64)
            assert tot[0::2].sum() + self.n_eq == self.k
            eq_before = int(tot[1:2 * self.index:2].sum())
            mine = max(0, min(int(tot[2 * self.index + 1]), self.n_eq - eq_before))
            eq_pos = np.flatnonzero(self.key == self.T)[:mine]
            idx = np.sort(np.concatenate([np.flatnonzero(self.key > self.T), eq_pos]))
            val = self.a[idx].copy()
            self.e = self.a.copy()
            self.e[idx] = 0.0
            self.slot = self.t % self.m
            self.rows[self.slot] = (idx, val)
            c = np.zeros(self.hi - self.lo)
            c[idx] = val
            self.buf[4][:] = torch.from_numpy(
                np.array([float(np.dot(v.astype(np.float64), c[i])) for i, v in self.rows]))
        else:
            delta = self.buf[4].numpy()
            self.S[self.slot, :] = delta
            self.S[:, self.slot] = delta
            lam = float(self.lam)
            rhs = np.zeros(self.m)
            rhs[self.slot] = self.m
            w = np.linalg.solve(self.m * lam * np.eye(self.m) + self.S, rhs)
            u = np.zeros(self.hi - self.lo)
            for wr, (i, v) in zip(w, self.rows):
                u[i] += wr * v.astype(np.float64)
            update.copy_(torch.from_numpy(u.astype(np.float32)))
            self.t += 1


def main():
    from oracle import ref
    from paper_2306_06098_b200 import sharded
    dist.init_process_group(backend="gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    d, m, k, lam, steps = 6000, 4, 61, 1e-2, 7
    ranges = sharded.even_ranges(d, world, align=1)
    lo, hi = ranges[rank]
    shard = NumpyShard(lo, hi, m, k, lam, rank, world)
    stepper = sharded.ShardedStep([shard], sharded.sum_over_processes())
    rng = np.random.default_rng(5)  # the same stream on every rank
    cpu = ref.RefEFCP(d, m, k, lam) if rank == 0 else None
    worst = 0.0
    ok = True
    for t in range(steps):
        # small integers: many ties at the threshold, on both sides of the shard boundary
        g = (rng.integers(-3, 4, d) * (1.0 if t % 2 else 0.5)).astype(np.float32)
        u_loc = torch.empty(hi - lo, dtype=torch.float32)
        stepper.step([torch.from_numpy(g[lo:hi].copy())], [u_loc])
        pieces = [None] * world
        dist.all_gather_object(pieces, (shard.e, shard.rows[t % m][0] + lo, shard.rows[t % m][1],
                                        u_loc.numpy()))
        if rank == 0:
            u_ref = cpu.step(g)
            e = np.concatenate([p[0] for p in pieces])
            i = np.concatenate([p[1] for p in pieces])
            v = np.concatenate([p[2] for p in pieces])
            u = np.concatenate([p[3] for p in pieces])
            ci, cv = cpu.row(t % m)
            ok &= np.array_equal(e.view(np.uint32), cpu.error().view(np.uint32))
            ok &= np.array_equal(i, ci) and np.array_equal(v.view(np.uint32), cv.view(np.uint32))
            worst = max(worst, float(np.linalg.norm(u - u_ref) / np.linalg.norm(u_ref)))
    order_ok = shard.calls == [(p, p == 0, p == 5) for _ in range(steps) for p in range(6)]
    print(json.dumps({"rank": rank, "world": world, "state_ok": bool(ok), "worst_u": worst,
                      "order_ok": order_ok}), flush=True)
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
