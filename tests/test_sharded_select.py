"""The select of one vector that is range-partitioned over several ranks (one small all-reduce per radix pass).

CPU part (gloo, world size 2): the rounds of the exchange -- per-rank digit histograms, their sum over the ranks, the
digit every rank derives from the sum -- with the per-rank pieces restated in numpy on the oracle's key order; both
ranks must arrive at the oracle's select of the concatenated vector.
GPU part: the library's kernels for the per-rank pieces, the ranks emulated one after the other on one GPU (the
histograms are summed by hand; nothing waits for anything), against the oracle and against dct_threshold_select."""
import os
import sys

import numpy as np
import pytest
import torch

import oracle
from paper_2010_08899_b200 import inputs
from tests._util import bits32

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SHIFT, BITS = (20, 10, 0), (11, 10, 10)


class _NumpyShard:
    """One rank's pieces of the radix select on its shard, on the oracle's total order key(x) = bits(x) & 0x7FFFFFFF."""

    def __init__(self, w: np.ndarray, k: int):
        self.keys = w.view(np.uint32) & np.uint32(0x7FFFFFFF)
        self.prefix, self.k_rem, self.n_gt, self.n_eq = 0, k, 0, 0

    def histogram(self, p: int) -> np.ndarray:
        keys = self.keys if p == 0 else self.keys[(self.keys >> np.uint32(SHIFT[p] + BITS[p])) == self.prefix]
        return np.bincount(((keys >> np.uint32(SHIFT[p])) & np.uint32((1 << BITS[p]) - 1)).astype(np.int64),
                           minlength=2048).astype(np.int64)

    def advance(self, p: int, hist: np.ndarray) -> None:
        above = 0
        for digit in range(2047, -1, -1):                       # from the top: the digit that holds rank k_rem
            c = int(hist[digit])
            if above < self.k_rem <= above + c:
                self.prefix = (self.prefix << BITS[p]) | digit
                self.k_rem -= above
                self.n_gt += above
                self.n_eq = c
                return
            above += c
        raise AssertionError("k exceeds the number of elements")

    @property
    def tau(self) -> np.float32:
        return np.array([self.prefix], np.uint32).view(np.float32)[0]


def _worker(rank, world, port, n, k, q):
    import torch.distributed as dist
    from paper_2010_08899_b200 import binding as B
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    g = inputs.quantize_mantissa(inputs.dp_gaussian(n, 5), 8).numpy()      # the whole vector (same seed everywhere)
    lo, hi = rank * n // world + (3 if rank else 0), (rank + 1) * n // world + (3 if rank + 1 < world else 0)
    shard = _NumpyShard(g[lo:hi], k)

    def all_reduce_sum(h):
        t = torch.from_numpy(h)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return t.numpy()

    B.sharded_select_rounds(shard.histogram, shard.advance, all_reduce_sum)
    q.put((rank, int(np.float32(shard.tau).view(np.uint32)), shard.n_gt, shard.n_eq))
    dist.destroy_process_group()


def test_rounds_of_the_sharded_select_on_two_gloo_ranks():
    import torch.multiprocessing as mp
    n, k, world = 50_000, 777, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, world, port, n, k, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    want = oracle.dp_select(inputs.quantize_mantissa(inputs.dp_gaussian(n, 5), 8).numpy(), None, k)
    for rank, tau_bits, n_gt, n_eq in got:
        assert tau_bits == int(bits32(want.tau)[0]) and (n_gt, n_eq) == (want.n_gt, want.n_eq), rank


def test_numpy_shard_restates_the_oracle_on_one_rank():
    g = inputs.dp_gaussian(20_001, 6).numpy()
    for k in (1, 2, 500, 20_001):
        s = _NumpyShard(g, k)
        for p in range(3):
            s.advance(p, s.histogram(p))
        want = oracle.dp_select(g, None, k)
        assert bits32(s.tau)[0] == bits32(want.tau)[0] and (s.n_gt, s.n_eq) == (want.n_gt, want.n_eq)


@pytest.mark.gpu
@pytest.mark.parametrize("ranks", [1, 3, 8])
def test_gpu_shard_kernels_against_the_oracle(ranks):
    from paper_2010_08899_b200 import binding as B
    n = (1 << 21) + 12_345
    g = inputs.quantize_mantissa(inputs.dp_mixture(n, 7, "cuda"), 9)         # ties at the threshold are likely
    e = inputs.dp_gaussian(n, 8, "cuda") * 0.01
    # uneven shards, one of them empty, none on a 16-byte boundary except the first
    cuts = sorted({0, n} | {int(n * f) + 1 for f in np.linspace(0, 1, ranks + 1)[1:-1]})
    if ranks > 2:
        cuts.insert(2, cuts[1])                                               # an empty shard
    shards = list(zip(cuts[:-1], cuts[1:]))
    L, s = B.lib(), torch.cuda.current_stream().cuda_stream
    for k in (1, 1000, n // 3, n):
        states = [B.new_workspace(B.dct_threshold_select_shard_workspace_bytes()) for _ in shards]
        taus = [torch.zeros(1, device="cuda") for _ in shards]
        results = [B.new_result() for _ in shards]
        hists = [torch.empty(2048, dtype=torch.int64, device="cuda") for _ in shards]
        for st in states:
            assert L.dct_threshold_select_shard_begin(k, st.data_ptr(), st.numel(), s) == 0
        for p in range(3):
            for (lo, hi), st, h in zip(shards, states, hists):
                gs, es = g[lo:hi], e[lo:hi]
                assert L.dct_threshold_select_shard_pass(gs.data_ptr() if hi > lo else None, es.data_ptr() if hi > lo else None,
                                                         hi - lo, p, st.data_ptr(), h.data_ptr(), s) == 0
            total = torch.stack(hists).sum(0)                                 # what the all-reduce would deliver
            for st, tau, res in zip(states, taus, results):
                assert L.dct_threshold_select_shard_advance(total.data_ptr(), p, st.data_ptr(), tau.data_ptr(),
                                                            res.data_ptr(), s) == 0
        want = oracle.dp_select(g.cpu().numpy(), e.cpu().numpy(), k)
        for tau, res in zip(taus, results):
            r = B.read_result(res)
            assert bits32(tau.cpu().numpy())[0] == bits32(want.tau)[0]
            assert (r.n_gt, r.n_eq, r.status) == (want.n_gt, want.n_eq, B.DCT_OK)


@pytest.mark.gpu
def test_gpu_sharded_select_through_the_binding_on_one_rank():
    from paper_2010_08899_b200 import binding as B
    n, k = 3_000_001, 4321
    g = inputs.dp_mixture(n, 9, "cuda")
    tau, res = torch.zeros(1, device="cuda"), B.new_result()
    B.dct_threshold_select_sharded(g, None, n, k, tau, res, B.new_workspace(B.dct_threshold_select_shard_workspace_bytes()))
    tau1, res1 = torch.zeros(1, device="cuda"), B.new_result()
    B.dct_threshold_select(g, None, n, k, tau1, res1, B.new_workspace(B.dct_threshold_select_workspace_bytes(n)))
    a, b = B.read_result(res), B.read_result(res1)
    assert torch.equal(tau, tau1) and (a.n_gt, a.n_eq) == (b.n_gt, b.n_eq)


# ---- the sampled variant: six rounds, one streaming pass over the shard ---------------------------------------------

class _NumpySampledShard(_NumpyShard):
    """One rank's pieces of the sampled rounds: two passes over a strided sample (the same stride on every rank),
    the filter (keys >= lo; the message is [count, overflowed]), and three passes over the candidates or, if the
    summed message says that they are too few or did not fit somewhere, over the shard."""

    def __init__(self, w: np.ndarray, k: int, n_global: int, sample_target: int, capacity: int):
        super().__init__(w, k)
        self.stride = max(8, (n_global // (sample_target // 8)) & ~7)
        rate = 8.0 / self.stride
        m = k * rate
        self.sample = _NumpyShard(self._sample_of(w), int(m + 6.0 * np.sqrt(m + 1.0) + 20.0))
        self.capacity, self.cand, self.use_cand = capacity, None, False

    def _sample_of(self, w):
        n = len(w)
        groups = (n - 8) // self.stride + 1 if n >= 8 else 0
        idx = (np.arange(groups)[:, None] * self.stride + np.arange(8)[None, :]).reshape(-1)
        return w[idx]

    def counts(self, r: int) -> np.ndarray:
        if r < 2:
            return self.sample.histogram(r)
        if r == 2:
            lo = self.sample.prefix << 10
            self.cand = self.keys[self.keys >= lo]
            msg = np.zeros(2048, np.int64)
            msg[0], msg[1] = len(self.cand), int(len(self.cand) > self.capacity)
            return msg
        src = _NumpyShard.__new__(_NumpyShard)
        src.keys, src.prefix = (self.cand if self.use_cand else self.keys), self.prefix
        return src.histogram(r - 3)

    def act(self, r: int, summed: np.ndarray) -> None:
        if r < 2:
            self.sample.advance(r, summed)
        elif r == 2:
            self.use_cand = summed[1] == 0 and summed[0] >= self.k_rem
        else:
            self.advance(r - 3, summed)


def _sampled_worker(rank, world, port, n, k, mode, q):
    import torch.distributed as dist
    from paper_2010_08899_b200 import binding as B
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    g = _sampled_case(n, mode)
    if mode == "plain":
        lo, hi = rank * n // world + (3 if rank else 0), (rank + 1) * n // world + (3 if rank + 1 < world else 0)
    else:       # the shards start on multiples of the stride, so that every rank's sample looks where the case expects
        stride = max(8, (n // ((1 << 12) // 8)) & ~7)
        cut = (n // world) // stride * stride
        lo, hi = rank * cut, (n if rank + 1 == world else (rank + 1) * cut)
    shard = _NumpySampledShard(g[lo:hi], k, n, sample_target=1 << 12, capacity=4000)

    def all_reduce_sum(h):
        t = torch.from_numpy(h)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return t.numpy()

    B.sharded_select_rounds(shard.counts, shard.act, all_reduce_sum, rounds=B.SHARD_SAMPLED_ROUNDS)
    q.put((rank, int(np.float32(shard.tau).view(np.uint32)), shard.n_gt, shard.n_eq, bool(shard.use_cand)))
    dist.destroy_process_group()


def _sampled_case(n, mode):
    """plain: the sample is representative.  hidden: the large values sit where the sample never looks (far too
    many candidates: they do not fit).  lure: the large values sit only where the sample looks (too few)."""
    g = inputs.quantize_mantissa(inputs.dp_gaussian(n, 5), 8).numpy().copy()
    if mode != "plain":
        stride = max(8, (n // ((1 << 12) // 8)) & ~7)
        on_sample = (np.arange(n) % stride) < 8
        g[on_sample if mode == "hidden" else ~on_sample] *= np.float32(1e-3)
    return g


@pytest.mark.parametrize("mode,uses_candidates", [("plain", True), ("hidden", False), ("lure", False)])
def test_rounds_of_the_sampled_sharded_select_on_two_gloo_ranks(mode, uses_candidates):
    import torch.multiprocessing as mp
    n, k, world = 200_000, 777, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000 + {"plain": 0, "hidden": 1, "lure": 2}[mode]
    procs = [ctx.Process(target=_sampled_worker, args=(r, world, port, n, k, mode, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    want = oracle.dp_select(_sampled_case(n, mode), None, k)
    for rank, tau_bits, n_gt, n_eq, used in got:
        assert tau_bits == int(bits32(want.tau)[0]) and (n_gt, n_eq) == (want.n_gt, want.n_eq), rank
        assert used == uses_candidates


@pytest.mark.gpu
@pytest.mark.parametrize("ranks", [1, 3, 8])
@pytest.mark.parametrize("mode", ["plain", "hidden", "lure"])
def test_gpu_sampled_shard_kernels_against_the_oracle(ranks, mode):
    """The library's sampled rounds with the ranks emulated one after the other on one GPU (the messages are summed by
    hand): a representative sample, and the two ways a sample can misjudge the vector (candidates overflow a rank's
    buffer / fewer candidates than k), which must end in the three passes over the shards with the same result."""
    from paper_2010_08899_b200 import binding as B
    n = (1 << 25) + 12_345
    g = inputs.quantize_mantissa(inputs.dp_mixture(n, 7, "cuda"), 9)         # ties at the threshold are likely
    e = inputs.dp_gaussian(n, 8, "cuda") * 0.01
    stride = (n // ((1 << 20) // 8)) & ~7
    if mode != "plain":
        # groups are taken at multiples of the stride inside every shard: only the first shard's positions are known
        # here, so the first shard gets (nearly) all of the vector
        on_sample = (torch.arange(n, device="cuda") % stride) < 8
        keep = on_sample if mode == "lure" else ~on_sample
        g = torch.where(keep, g, g * 1e-3)
        e = torch.where(keep, e, e * 1e-3)
        cuts = [0, n - 64 * (ranks - 1)] + [n - 64 * (ranks - 1 - i) for i in range(1, ranks)]
    else:
        cuts = sorted({0, n} | {int(n * f) + 1 for f in np.linspace(0, 1, ranks + 1)[1:-1]})
        if ranks > 2:
            cuts.insert(2, cuts[1])                                           # an empty shard
    shards = list(zip(cuts[:-1], cuts[1:]))
    L, s = B.lib(), torch.cuda.current_stream().cuda_stream
    k = 20_000
    states = [B.new_workspace(B.dct_threshold_select_shard_sampled_workspace_bytes(hi - lo)) for lo, hi in shards]
    taus = [torch.zeros(1, device="cuda") for _ in shards]
    results = [B.new_result() for _ in shards]
    hists = [torch.empty(2048, dtype=torch.int64, device="cuda") for _ in shards]
    for (lo, hi), st in zip(shards, states):
        assert L.dct_threshold_select_shard_sampled_begin(k, n, hi - lo, st.data_ptr(), st.numel(), s) == 0
    used = None
    for r in range(B.SHARD_SAMPLED_ROUNDS):
        for (lo, hi), st, h in zip(shards, states, hists):
            gs, es = g[lo:hi], e[lo:hi]
            assert L.dct_threshold_select_shard_sampled_pass(gs.data_ptr() if hi > lo else None,
                                                             es.data_ptr() if hi > lo else None, hi - lo, r,
                                                             st.data_ptr(), h.data_ptr(), s) == 0
        total = torch.stack(hists).sum(0)                                     # what the all-reduce would deliver
        if r == 2:
            used = int(total[1]) == 0 and int(total[0]) >= k
        for st, tau, res in zip(states, taus, results):
            assert L.dct_threshold_select_shard_sampled_advance(total.data_ptr(), r, st.data_ptr(), tau.data_ptr(),
                                                                res.data_ptr(), s) == 0
    assert used == (mode == "plain")
    want = oracle.dp_select(g.cpu().numpy(), e.cpu().numpy(), k)
    for tau, res in zip(taus, results):
        rr = B.read_result(res)
        assert bits32(tau.cpu().numpy())[0] == bits32(want.tau)[0]
        assert (rr.n_gt, rr.n_eq, rr.status) == (want.n_gt, want.n_eq, B.DCT_OK)


@pytest.mark.gpu
def test_gpu_sampled_sharded_select_through_the_binding_on_one_rank():
    from paper_2010_08899_b200 import binding as B
    n, k = (1 << 25) + 77, 54_321
    g = inputs.dp_mixture(n, 9, "cuda")
    tau, res = torch.zeros(1, device="cuda"), B.new_result()
    ws = B.new_workspace(B.dct_threshold_select_shard_sampled_workspace_bytes(n))
    assert B.dct_threshold_select_sharded(g, None, n, k, tau, res, ws, n_global=n) is True
    tau1, res1 = torch.zeros(1, device="cuda"), B.new_result()
    B.dct_threshold_select(g, None, n, k, tau1, res1, B.new_workspace(B.dct_threshold_select_workspace_bytes(n)))
    a, b = B.read_result(res), B.read_result(res1)
    assert torch.equal(tau, tau1) and (a.n_gt, a.n_eq) == (b.n_gt, b.n_eq)
    # too small a vector, or too dense a k: the three-pass rounds run instead
    assert B.dct_threshold_select_sharded(g[:1 << 20], None, 1 << 20, 100, tau, res, ws, n_global=1 << 20) is False
    assert B.dct_threshold_select_sharded(g, None, n, n // 3, tau, res, ws, n_global=n) is False
    B.dct_threshold_select(g, None, n, n // 3, tau1, res1, B.new_workspace(B.dct_threshold_select_workspace_bytes(n)))
    a, b = B.read_result(res), B.read_result(res1)
    assert torch.equal(tau, tau1) and (a.n_gt, a.n_eq) == (b.n_gt, b.n_eq)
