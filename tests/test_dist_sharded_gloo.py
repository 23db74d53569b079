"""The exchanges of the sharded-row solver between PROCESSES, on CPU: two gloo ranks, two shards each.

dist.forward_sharded / backward_sharded only need shard objects with the per-shard steps and the exchange tensors.
Here the steps are stand-ins written in numpy (with the oracle's seeded solve for the merged band): what is under
test is the orchestration - the key-buffer sum, the sums of tails / counts / tables, the concatenation of the bands
across ranks in row order, the sum of the VJP sums, and the whole-row fallback after a failed certificate.  The
assembled mask and gradient must be those of the oracle on the unsharded row."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

from oracle import lapsum_oracle as O
from paper_2608_06912_b200 import dist as D


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _keys(x):
    """order-preserving uint32 keys of fp32 values, as int32 bit patterns (what the exchange buffers hold)"""
    b = np.asarray(x, dtype=np.float32).view(np.uint32)
    u = np.where(b & 0x80000000, ~b, b | 0x80000000).astype(np.uint32)
    return u.view(np.int32)


def _floats(k):
    u = np.asarray(k).view(np.uint32)
    b = np.where(u & 0x80000000, u & 0x7FFFFFFF, ~u).astype(np.uint32)
    return b.view(np.float32)


class FakeShard:
    """CPU stand-in for binding.GpuShard (test infrastructure: numpy + the oracle's routines)"""

    def __init__(self, r_shard, begin, n_total, seed, z=5.16, cap=4096):
        self.r = torch.from_numpy(np.ascontiguousarray(r_shard, dtype=np.float32))
        self.begin, self.n_total, self.len, self.seed, self.z = begin, n_total, len(r_shard), seed, z
        self.K = O.sample_count(n_total)
        self.band_capacity = cap
        self.sample_keys = torch.zeros(self.K, dtype=torch.int32)
        self.band_count = torch.zeros(1, dtype=torch.int64)
        self.n_R = torch.zeros(1, dtype=torch.int64)
        self.tails = torch.zeros(2, dtype=torch.float64)
        self.bucket_counts = torch.zeros(1024, dtype=torch.int32)
        self.bucket_sums = torch.zeros(2048, dtype=torch.int64)
        self.band_keys = torch.zeros(cap, dtype=torch.int32)
        self.vjp_sums = torch.zeros(4, dtype=torch.float64)
        self.b = torch.full((1,), float("nan"), dtype=torch.float64)
        self.p = torch.zeros(self.len)
        self.grad = torch.zeros(self.len)
        self.grad_k, self.grad_alpha = torch.zeros(1), torch.zeros(1)

    def sample(self, alpha):
        idx = O.sample_indices(self.seed, self.n_total, self.K)
        noise = O.noise_table(self.seed, self.K)
        mine = (idx >= self.begin) & (idx < self.begin + self.len)
        y = np.zeros(self.K, np.float32)
        r = self.r.numpy()
        y[mine] = (np.float32(abs(alpha)) * noise[mine].astype(np.float64) + r[idx[mine] - self.begin].astype(np.float64)).astype(np.float32)
        keys = np.zeros(self.K, np.int32)
        keys[mine] = _keys(y[mine])
        self.sample_keys.copy_(torch.from_numpy(keys))

    def stream_pass(self, k, alpha):
        t = abs(alpha)
        y = np.sort(_floats(self.sample_keys.numpy()))
        K, j, l = O.bracket_indices(self.n_total, k, self.z)
        self.a_L = float(y[j - 1]) if j >= 1 else -np.inf
        self.a_R = float(y[l - 1]) if l <= K else np.inf
        r = self.r.numpy().astype(np.float64)
        below, above = r < self.a_L, r >= self.a_R
        band = self.r.numpy()[~below & ~above]
        self.tails[0] = float(np.exp((r[below] - self.a_L) / t).sum())
        self.tails[1] = float(np.exp(-(r[above] - self.a_R) / t).sum())
        self.n_R[0] = int(above.sum())
        self.band_count[0] = len(band)
        m = min(len(band), self.band_capacity)
        self.band_keys[:m] = torch.from_numpy(_keys(band[:m]))

    def solve(self, k, alpha):
        m = int(self.band_count.item())
        if m > self.band_capacity:
            self.b[0] = float("nan")
            return
        band = np.sort(_floats(self.band_keys[:m].numpy())).astype(np.float64)
        res = O.solve_sorted(band, k, abs(alpha), self.a_L, float(self.tails[0]), self.a_R, float(self.tails[1]),
                             int(self.n_R.item()))
        self.b[0] = float("nan") if res.status else res.b

    def _cdf(self, x, b, t):
        u = (x - b) / t
        return np.where(u <= 0, 0.5 * np.exp(np.minimum(u, 0)), 1 - 0.5 * np.exp(-np.maximum(u, 0)))

    def mask(self, alpha):
        self.p.copy_(torch.from_numpy(self._cdf(self.r.numpy().astype(np.float64), float(self.b[0]), abs(alpha)).astype(np.float32)))

    def whole_row_forward(self, r_full, k, alpha):
        ref = O.forward(r_full.numpy().reshape(1, -1), k, alpha)
        self.b[0] = float(ref.b[0])
        self.p.copy_(torch.from_numpy(ref.p[0, self.begin:self.begin + self.len].astype(np.float32)))

    def _f(self, alpha):
        t = abs(alpha)
        d = self.r.numpy().astype(np.float64) - float(self.b[0])
        return np.exp(-np.abs(d) / t) / (2 * t), d

    def vjp_partial(self, v, alpha):
        f, d = self._f(alpha)
        v = v.numpy().astype(np.float64)
        self.vjp_sums.copy_(torch.tensor([f.sum(), (v * f).sum(), (f * d).sum(), (v * f * d).sum()], dtype=torch.float64))

    def vjp_apply(self, v, alpha):
        f, _ = self._f(alpha)
        S_f, S_vf, S_fd, S_vfd = self.vjp_sums.tolist()
        mean = S_vf / S_f
        self.grad.copy_(torch.from_numpy((f * (v.numpy().astype(np.float64) - mean)).astype(np.float32)))
        self.grad_k[0] = mean
        self.grad_alpha[0] = (S_vfd - mean * S_fd) / abs(alpha)


def _case(z):
    n, k, alpha, seed = 60_000, 900.0, -0.05, 12
    rng = np.random.default_rng(3)
    return n, k, alpha, seed, z, rng.standard_normal(n).astype(np.float32), rng.standard_normal(n).astype(np.float32)


def _worker(rank, world, port, z, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    D.init("gloo")
    n, k, alpha, seed, z, r, v = _case(z)
    half = n // world
    lo = rank * half
    cuts = [lo, lo + half // 3, lo + half]          # two unequal shards per rank, in row order
    shards = [FakeShard(r[a:b], a, n, seed, z) for a, b in zip(cuts[:-1], cuts[1:])]
    # every rank holds `half` scores, so the whole-row gather may use an equal-size collective
    held = D.forward_sharded(shards, k, alpha, gather_row=D.gather_row_over(shards))
    D.backward_sharded(shards, [torch.from_numpy(v[s.begin:s.begin + s.len]) for s in shards], alpha)
    out.put((rank, held, float(shards[0].b[0]), float(shards[1].b[0]), torch.cat([s.p for s in shards]).numpy(),
             torch.cat([s.grad for s in shards]).numpy(), float(shards[0].grad_k[0]), int(shards[0].band_count.item())))
    D.barrier()
    D.finalize()


def _run(z):
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, z, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=180) for _ in range(world)), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    return res


def _check(res, held_expected):
    n, k, alpha, seed, z, r, v = _case(5.16)
    ref = O.forward(r.reshape(1, -1), k, alpha)
    g_ref = O.backward(v.reshape(1, -1), r.reshape(1, -1), ref.b, alpha)[0]
    gk_ref, _ = O.backward_scalars(v.reshape(1, -1), r.reshape(1, -1), ref.b, alpha)
    assert [x[1] for x in res] == [held_expected] * 2
    for rank, held, b0, b1, p, g, gk, n_M in res:
        assert abs(b0 - ref.b[0]) <= 1e-9 and b0 == b1            # the same threshold on every shard of every rank
        assert abs(gk - gk_ref[0]) <= 1e-6
    p = np.concatenate([x[4] for x in res]).astype(np.float64)
    g = np.concatenate([x[5] for x in res]).astype(np.float64)
    assert np.max(np.abs(p - ref.p[0])) <= 1e-6 and abs(p.sum() - k) <= 1e-3
    assert np.max(np.abs(g - g_ref)) <= 1e-5 * np.max(np.abs(g_ref))
    assert res[0][7] == res[1][7]                                  # both ranks ended with the same merged band count
    return res


def test_two_ranks_two_shards_each_match_the_oracle():
    res = _check(_run(5.16), True)
    n, k, alpha, seed, z, r, v = _case(5.16)
    want = O.bracket(r.reshape(1, -1), k, alpha, 5.16, seed)
    assert res[0][7] == want.n_M                                   # the merged band is the unsharded row's band


def test_failed_certificate_ends_in_the_whole_row_forward_on_every_rank():
    # a bracket so narrow that it misses: z = 0.01 leaves (almost) no band around the sampled quantile
    _check(_run(0.01), False)
