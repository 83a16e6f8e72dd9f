"""The library's enqueue-only calls inside CUDA-graph capture (GPU).

A captured sequence of relayout, dense, grouped, expert-FFN and counter launches must replay with the bits of the
same calls issued directly, on whatever the input buffers hold at replay time.  Integer-valued inputs make the dense
and grouped products exact, so the replayed results are also compared with the exact integer product.
"""
import numpy as np
import pytest
import torch

import oracle as tlo
from paper_2607_04031_b200 import inputs

pytestmark = pytest.mark.gpu

G, BR, BC = 4096, 16, 128


def _products():
    # (M, N, K, forced cut): split-K inside clusters, whole tiles, and the stream-K cut (which needs scratch)
    # ... then a tile of two token blocks (128 tiles on 128 CTAs) and a product on CTA pairs
    return [(8, 1024, 4096, False), (16, 148 * 256, 256, False), (24, 1280, 2048, True), (1024, 8192, 256, False),
            (512, 19200, 128, False)]


class _Step:
    """Fixed buffers, one method that issues every call of the step on the current stream."""

    def __init__(self, tl, dev):
        self.tl, self.dev = tl, dev
        self.W_row, self.W_tile, self.A, self.C = [], [], [], []
        for M, N, K, _ in _products():
            self.W_row.append(torch.empty((K, N), dtype=torch.bfloat16, device=dev))
            self.W_tile.append(torch.empty((K, N), dtype=torch.bfloat16, device=dev))
            self.A.append(torch.empty((M, K), dtype=torch.bfloat16, device=dev))
            self.C.append(torch.empty((M, N), dtype=torch.float32, device=dev))
        # grouped product and expert FFN over one routing
        self.rows = np.array([5, 0, 40, 17, 33, 1, 0, 64], dtype=np.int64)
        self.E, self.total = len(self.rows), int(self.rows.sum())
        self.offs = np.concatenate([[0], np.cumsum(self.rows)]).astype(np.int32)
        self.d_offs = torch.from_numpy(self.offs).to(dev)
        self.hidden, self.inter = 512, 256
        self.X = torch.empty((self.total, self.hidden), dtype=torch.bfloat16, device=dev)
        self.Wg_row = torch.empty((self.E * self.hidden, 2 * self.inter), dtype=torch.bfloat16, device=dev)
        self.Wg = torch.empty_like(self.Wg_row)
        self.Wd_row = torch.empty((self.E * self.inter, self.hidden), dtype=torch.bfloat16, device=dev)
        self.Wd = torch.empty_like(self.Wd_row)
        self.Cg = torch.empty((self.total, 2 * self.inter), dtype=torch.float32, device=dev)
        self.H = torch.empty((self.total, self.inter), dtype=torch.bfloat16, device=dev)
        self.Y = torch.empty((self.total, self.hidden), dtype=torch.float32, device=dev)
        self.counts = torch.zeros((len(_products()), 3), dtype=torch.int64, device=dev)
        self.cfgs = tl.read_amp_cfgs((M, N, K, tl.gemm_plan(M, N, K, G, BR, BC).cta, tl.LAYOUT_TILE_MAJOR, G, BR, BC, 2)
                                     for M, N, K, _ in _products())
        # one workspace of the caller's for every launch of the step that needs scratch (they run one after the other):
        # two partial tiles of up to 128 x 256 floats per CTA
        self.ws = torch.empty(2 * 148 * 128 * 256 * 4, dtype=torch.uint8, device=dev)

    def load(self, seed):
        for i, (M, N, K, _) in enumerate(_products()):
            self.W_row[i].copy_(inputs.bf16_integers((K, N), -4, 4, seed=seed + 10 * i, device=self.dev))
            self.A[i].copy_(inputs.bf16_integers((M, K), -4, 4, seed=seed + 10 * i + 1, device=self.dev))
        self.X.copy_(inputs.bf16_integers(tuple(self.X.shape), -3, 3, seed=seed + 100, device=self.dev))
        self.Wg_row.copy_(inputs.bf16_integers(tuple(self.Wg_row.shape), -2, 2, seed=seed + 101, device=self.dev))
        self.Wd_row.copy_(inputs.bf16_integers(tuple(self.Wd_row.shape), -2, 2, seed=seed + 102, device=self.dev))

    def outputs(self):
        return [*self.C, self.Cg, self.H, self.Y, self.counts, *self.W_tile, self.Wg, self.Wd]

    def poison(self):
        for t in self.outputs():
            if t.dtype.is_floating_point:
                t.fill_(float("nan"))
            else:
                t.fill_(-1)

    def issue(self):
        self.tl.set_workspace(self.ws)
        try:
            self._issue()
        finally:
            self.tl.set_workspace(None)

    def _issue(self):
        tl = self.tl
        tl.relayout_batch(self.W_row, self.W_tile, [(K, N) for _, N, K, _ in _products()], 2, G, BR, BC, tl.TO_TILE_MAJOR)
        tl.relayout(self.Wg_row, self.Wg, self.E * self.hidden, 2 * self.inter, 2, G, BR, BC, tl.TO_TILE_MAJOR)
        tl.relayout(self.Wd_row, self.Wd, self.E * self.inter, self.hidden, 2, G, BR, BC, tl.TO_TILE_MAJOR)
        self.plans = []
        for i, (M, N, K, cut) in enumerate(_products()):
            if cut:
                with tl.option(tl.OPT_NO_SCRATCH_PLANS, 0):
                    tl.gemm(self.A[i], self.W_tile[i], self.C[i], M, N, K, G, BR, BC)
            else:
                tl.gemm(self.A[i], self.W_tile[i], self.C[i], M, N, K, G, BR, BC)
            self.plans.append(tl.gemm_last_plan())
        tl.gemm_grouped(self.X, self.Wg, self.Cg, self.d_offs, self.E, self.total, 2 * self.inter, self.hidden, G, BR, BC)
        tl.moe_ffn(self.X, self.Wg, self.Wd, self.H, self.Y, self.d_offs, self.E, self.total, self.hidden, self.inter,
                   G, BR, BC)
        tl.read_amp_batch(self.cfgs, self.counts)


def _same(a, b):
    if a.dtype.is_floating_point:
        return torch.equal(a.view(torch.int16 if a.element_size() == 2 else torch.int32),
                           b.view(torch.int16 if b.element_size() == 2 else torch.int32))
    return torch.equal(a, b)


def test_a_captured_step_replays_the_bits_of_direct_calls():
    from gpu_util import DEV, tl
    step = _Step(tl, DEV)
    want = {}
    for seed in (1, 2):                                   # direct calls on two input sets (also the warm-up)
        step.load(seed)
        step.poison()
        step.issue()
        tl.device_status()
        want[seed] = [t.clone() for t in step.outputs()]
    kinds = [(p.stream_k, p.cluster_k > 1) for p in step.plans[:3]]
    assert kinds == [(0, True), (0, False), (1, False)], kinds     # clusters, whole tiles, the cut
    assert step.plans[3].cta == (256, 256, 64) and step.plans[4].pair_kernel == 1
    # the dense and grouped products are exact integers
    for i, (M, N, K, _) in enumerate(_products()):
        exact = step.A[i].double() @ step.W_row[i].double()
        assert torch.equal(want[2][i].double(), exact)
    for e in range(step.E):
        a, b = step.offs[e], step.offs[e + 1]
        exact = step.X[a:b].double() @ step.Wg_row[e * step.hidden:(e + 1) * step.hidden].double()
        assert torch.equal(want[2][len(_products())][a:b].double(), exact)
    # the counters equal the oracle's brute force
    for i, (M, N, K, _) in enumerate(_products()):
        cta = step.plans[i].cta
        fetched, used, _req = tlo.read_amp(M, N, K, cta[0], cta[1], cta[2], tlo.TILE_MAJOR, G, BR, BC, 2)
        assert tuple(int(x) for x in want[2][len(_products()) + 3][i][:2].cpu()) == (fetched, used)

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step.issue()
    for seed in (1, 2, 1):
        step.load(seed)
        step.poison()
        graph.replay()
        tl.device_status()
        for got, ref in zip(step.outputs(), want[seed]):
            assert _same(got, ref), seed


def test_a_captured_launch_takes_scratch_only_from_the_callers_workspace():
    from gpu_util import DEV, tl
    M, N, K = 24, 1280, 2048
    A = inputs.bf16_integers((M, K), -4, 4, seed=5, device=DEV)
    W = inputs.bf16_integers((K, N), -4, 4, seed=6, device=DEV)
    Wt = torch.empty_like(W)
    tl.relayout(W, Wt, K, N, 2, G, BR, BC, tl.TO_TILE_MAJOR)
    C = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
    with tl.option(tl.OPT_NO_SCRATCH_PLANS, 0):
        tl.gemm(A, Wt, C, M, N, K, G, BR, BC)            # warm-up; the internal workspace exists and is large enough
        assert tl.gemm_last_plan().stream_k == 1
        tl.device_status()
        graph = torch.cuda.CUDAGraph()
        refused = None
        with torch.cuda.graph(graph):
            try:
                tl.gemm(A, Wt, C, M, N, K, G, BR, BC)    # needs scratch, none of the caller's: refused, nothing enqueued
            except tl.TileLensError as e:
                refused = e.status
            with tl.option(tl.OPT_NO_SCRATCH_PLANS, 1):
                tl.gemm(A, Wt, C, M, N, K, G, BR, BC)    # the capture is still good: a schedule without scratch
                assert tl.gemm_last_plan().stream_k == 0
    assert refused == 6                                   # TL_ERR_WORKSPACE
    C.fill_(float("nan"))
    graph.replay()
    tl.device_status()
    assert torch.equal(C.double(), A.double() @ W.double())


def test_the_expert_ffn_runs_as_two_launches_while_captured():
    from gpu_util import DEV, tl
    step = _Step(tl, DEV)
    step.load(3)
    step.issue()
    tl.device_status()
    H0, Y0 = step.H.clone(), step.Y.clone()
    tl.set_workspace(step.ws)
    for form in (1, 2):
        with tl.option(tl.OPT_FFN_ONE_LAUNCH, form):
            tl.moe_ffn(step.X, step.Wg, step.Wd, step.H, step.Y, step.d_offs, step.E, step.total, step.hidden, step.inter,
                       G, BR, BC)                         # warm-up of the one-launch form outside any capture
            tl.device_status()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                tl.moe_ffn(step.X, step.Wg, step.Wd, step.H, step.Y, step.d_offs, step.E, step.total, step.hidden,
                           step.inter, G, BR, BC)
                assert tl.gemm_last_plan().chained == 0
        step.H.fill_(float("nan"))
        step.Y.fill_(float("nan"))
        graph.replay()
        graph.replay()
        tl.device_status()
        assert _same(step.H, H0) and _same(step.Y, Y0), form
    tl.set_workspace(None)
