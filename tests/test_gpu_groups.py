"""Groups of independent layers enqueued side by side (the query / key / value projections of an attention block):
parity of every layer with the oracle, agreement with the single-layer calls, replay from a CUDA graph (same bits
every time), and the argument checks that run before anything is enqueued."""
import numpy as np
import pytest
import torch

from paper_2309_03824_b200 import binding as b
from paper_2309_03824_b200 import workloads as wl

from helpers import DT, TOL, dev, host, oracle_linear, rel_err, run_linear, workspace

pytestmark = pytest.mark.gpu

NAMES = ("Y", "Z", "dX", "dU", "dV", "db")


def make_group(shapes, seed, shared_x=False):
    cases = [wl.random_factor_case(M, K, N, r, "bf16", seed + 7 * i) for i, (M, K, N, r) in enumerate(shapes)]
    if shared_x:
        for c in cases[1:]:
            c["X"] = cases[0]["X"]
    return cases


class Group:
    def __init__(self, cases, freeze):
        code, tdt = DT["bf16"]
        self.cases, self.freeze, self.n = cases, freeze, len(cases)
        self.descs = [b.linear_desc(c["M"], c["K"], c["N"], c["r"], code) for c in cases]
        self.in_ = {k: [dev(c[k], "bf16") for c in cases] for k in ("X", "V", "U", "b", "dY")}
        nan = float("nan")
        self.out = {"Y": [torch.full((c["M"], c["N"]), nan, dtype=tdt, device="cuda") for c in cases],
                    "Z": None if freeze == b.LRD_FREEZE_U else [torch.full((c["M"], c["r"]), nan, dtype=tdt, device="cuda") for c in cases],
                    "dX": [torch.full((c["M"], c["K"]), nan, dtype=tdt, device="cuda") for c in cases],
                    "dU": [torch.full((c["N"], c["r"]), nan, dtype=tdt, device="cuda") for c in cases],
                    "dV": [torch.full((c["K"], c["r"]), nan, dtype=tdt, device="cuda") for c in cases],
                    "db": [torch.full((c["N"],), nan, dtype=tdt, device="cuda") for c in cases]}
        self.ws = [workspace(max(b.lrd_linear_workspace_bytes(d, freeze, 0), b.lrd_linear_workspace_bytes(d, freeze, 1))) for d in self.descs]

    def fwd(self):
        i, o_ = self.in_, self.out
        b.lrd_linear_group_fwd(self.descs, i["X"], i["V"], i["U"], i["b"], o_["Y"], o_["Z"], self.freeze, self.ws)

    def bwd(self):
        i, o_ = self.in_, self.out
        b.lrd_linear_group_bwd(self.descs, i["dY"], None if self.freeze == b.LRD_FREEZE_V else i["X"], i["V"], i["U"], o_["Z"],
                               o_["dX"], o_["dU"], o_["dV"], o_["db"], self.freeze, self.ws)

    def check(self, single=True):
        torch.cuda.synchronize()
        assert b.lrd_check_device_status() == b.LRD_OK
        for li, case in enumerate(self.cases):
            ref = oracle_linear(case, self.freeze)
            one = run_linear(case, self.freeze) if single else None
            for name in NAMES:
                if self.out[name] is None:
                    continue
                got = self.out[name][li]
                assert rel_err(got, ref[name]) <= TOL["bf16"], (li, name)
                # A group changes where and beside what a layer runs.  The intermediate has the bits of a single-layer
                # call; the second product of a chain walks over the rank in an order that depends on the cluster size,
                # and the weight gradients of a group reduce over the tokens in fewer, larger shares, so Y, dX and
                # the weight gradients agree to rounding only.
                if one is not None and one[name] is not None:
                    if name == "Z":
                        assert torch.equal(got, one[name]), (li, name)
                    else:
                        assert rel_err(got, host(one[name])) <= 2.0 ** -7, (li, name)


QKV = [(520, 264, 264, 64)] * 3
MIXED = [(300, 200, 136, 48), (300, 200, 520, 128), (700, 136, 200, 64), (130, 776, 72, 32)]


@pytest.mark.parametrize("freeze", [b.LRD_FREEZE_NONE, b.LRD_FREEZE_U, b.LRD_FREEZE_V])
@pytest.mark.parametrize("shapes,shared", [(QKV, True), (MIXED, False), ([(400, 328, 264, 96)], False)])
def test_group_matches_oracle_and_single_layer_calls(freeze, shapes, shared):
    g = Group(make_group(shapes, 1200 + len(shapes), shared), freeze)
    g.fwd()
    g.bwd()
    g.check()


def test_group_of_eight_layers_and_empty_group():
    g = Group(make_group([(260, 136, 136, 32)] * 8, 1300), b.LRD_FREEZE_NONE)
    g.fwd()
    g.bwd()
    g.check(single=False)
    assert b.lrd_linear_group_fwd([], [], [], [], [], [], [], b.LRD_FREEZE_NONE, []) == b.LRD_OK


def test_group_replayed_from_a_cuda_graph():
    """Captured once (the side streams join the capture and rejoin before it ends), replayed on fresh outputs."""
    g = Group(make_group(QKV, 1400, shared_x=True), b.LRD_FREEZE_NONE)
    g.fwd()
    g.bwd()
    torch.cuda.synchronize()
    first = {k: [t.clone() for t in v] for k, v in g.out.items()}
    side, graph = torch.cuda.Stream(), torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            g.fwd()
            g.bwd()
    for _ in range(3):
        for v in g.out.values():
            for t in v:
                t.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        for k, v in g.out.items():
            for li, t in enumerate(v):
                assert torch.equal(t, first[k][li]), (k, li)
    g.check(single=False)


def test_group_checks_every_layer_before_enqueueing_anything():
    g = Group(make_group(QKV, 1500), b.LRD_FREEZE_U)
    good_ws = g.ws
    g.ws = [good_ws[0], good_ws[1], torch.empty(256, dtype=torch.uint8, device="cuda")]      # last layer: workspace too small
    outs = [t for v in g.out.values() if v is not None for t in v]
    for t in outs:
        t.fill_(7.0)
    with pytest.raises(b.LrdError):
        g.fwd()
    with pytest.raises(b.LrdError):
        g.bwd()
    torch.cuda.synchronize()
    for t in outs:
        assert bool((t == 7.0).all())              # the valid layers before it did not run either
    g.ws = good_ws
    with pytest.raises(b.LrdError):               # more layers than a group may hold
        big = Group(make_group([(130, 64, 64, 16)] * 9, 1600), b.LRD_FREEZE_U)
        big.fwd()
    with pytest.raises(ValueError):               # a per-layer list of the wrong length
        b.lrd_linear_group_fwd(g.descs, g.in_["X"][:2], g.in_["V"], g.in_["U"], g.in_["b"], g.out["Y"], g.out["Z"], g.freeze, g.ws)
    g.fwd()
    g.bwd()
    g.check(single=False)


def _svd_factors(W, r):
    Uf, s, Vt = np.linalg.svd(W, full_matrices=False)     # input construction only
    root = np.sqrt(s[:r])
    return Vt[:r].T * root, Uf[:, :r] * root


@pytest.mark.parametrize("freeze", [b.LRD_FREEZE_U, b.LRD_FREEZE_V])
def test_bert_base_attention_projections_as_the_benchmark_launches_them(freeze):
    """attn_q / attn_k / attn_v at full size (4096 tokens, 768 -> 768, r = 192, factors from an SVD) as one group:
    the launch configuration of the benchmark step, every output element against the oracle."""
    cases = []
    for idx, (name, K, N, r) in enumerate(wl.C1_BERT_LAYERS[:3]):
        cases.append(wl.linear_case(wl.C1_M, K, N, r, "bf16", 1000 + 10 * idx, wl.W_STD_TRANSFORMER, _svd_factors))
    g = Group(cases, freeze)
    g.fwd()
    g.bwd()
    g.check(single=False)


def test_groups_from_two_host_threads_at_once():
    """Every host thread has its own library streams: two threads, each with its own stream, run groups at the same
    time (the C calls release the interpreter lock), many times over; each must get its own right answers."""
    import threading
    gs = [Group(make_group(QKV, 1700 + 50 * t, shared_x=True), b.LRD_FREEZE_NONE) for t in range(2)]
    errors = []

    def work(g):
        try:
            st = torch.cuda.Stream()
            with torch.cuda.stream(st):
                for _ in range(20):
                    g.fwd()
                    g.bwd()
            st.synchronize()
        except Exception as e:          # surfaced in the main thread below
            errors.append(e)

    threads = [threading.Thread(target=work, args=(g,)) for g in gs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for g in gs:
        g.check(single=False)
