"""GPU parity of the model variants the paper's experiments use (Sec. 4.1 "GNN Encoders"): GCN
layers with the renormalised adjacency, PReLU, Layer Normalization before the activation -- every
combination, against the fp64 oracle on the same seeded inputs, at the tolerances of the base
model (1e-4 activations, 1e-3 gradients and parameters)."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2305_09887_b200 import inputs

pytestmark = pytest.mark.gpu

VARIANTS = [v for v in itertools.product((0, 1), (0, 1), (0, 1)) if v != (0, 0, 0)]


@pytest.fixture(scope="module")
def util():
    import gpu_util
    return gpu_util


def _start(variant, dims, seed):
    p = oracle.variant_init_params(variant, dims, seed)
    rng = np.random.default_rng(seed + 1)
    for lay in oracle.variant_layout(variant, dims):       # gamma, beta, slope away from 1, 0, 0.25
        for key, spread in (("gamma", 0.2), ("beta", 0.2), ("slope", 0.05)):
            if lay[key] >= 0:
                size = 1 if key == "slope" else dims[oracle.variant_layout(variant, dims).index(lay) + 1]
                p[lay[key]:lay[key] + size] += spread * rng.standard_normal(size)
    return p.astype(np.float32)


@pytest.mark.parametrize("variant", VARIANTS)
def test_variant_on_tiny(util, tiny_workload, variant):
    w = tiny_workload
    p0 = _start(variant, w.dims, 7)
    got, want = util.check_one_step(w, variant=variant, params0=p0)
    util.check_k_steps_and_average(w, got, want, 3, variant=variant, params0=p0)


@pytest.mark.parametrize("variant", [(1, 1, 1), (0, 1, 1)])
def test_variant_three_layers_power_law(util, variant):
    # the paper's encoder (PReLU + LayerNorm) on the Medium shape, scaled: several row tiles per
    # part, hubs, isolated local nodes
    w = inputs.medium(0.04)
    p0 = _start(variant, w.dims, 11)
    got, want = util.check_one_step(w, variant=variant, params0=p0)
    util.check_k_steps_and_average(w, got, want, 2, variant=variant, params0=p0)


@pytest.mark.parametrize("dims", [(6, 5, 3), (17, 130, 7, 2), (20, 300, 4)])
def test_gcn_prelu_layernorm_odd_widths(util, dims):
    w = inputs.tiny()
    w.dims = dims
    w.X = inputs.normal_features(w.graph.n, dims[0], 3)
    w.y = inputs.uniform_labels(w.graph.n, dims[-1], 4)
    p0 = _start((1, 1, 1), dims, 13)
    got, want = util.check_one_step(w, M=3, variant=(1, 1, 1), params0=p0)
    util.check_k_steps_and_average(w, got, want, 2, variant=(1, 1, 1), params0=p0)


@pytest.mark.parametrize("variant,dims", [((0, 0, 0), (64, 64, 2)), ((0, 0, 0), (24, 96, 1)), ((0, 0, 0), (64, 64, 3)),
                                          ((1, 0, 0), (64, 64, 4)), ((1, 0, 0), (40, 200, 2)), ((0, 0, 0), (32, 64, 48, 2)),
                                          ((0, 1, 1), (64, 64, 2))])
def test_heads_with_very_few_classes(util, variant, dims):
    # Few classes take paths of their own: the last layer aggregated after its product at class width by one
    # thread per row, its input gradient on the plain ALUs (up to 4 classes), and -- in a two-layer model with
    # at most 4 products per output and no separate activation pass -- generated inside the weight-gradient
    # kernel of the first layer instead of being written and read.  GraphSAGE (two weight matrices) and GCN
    # (one), one to four classes, two and three layers, a PReLU + LayerNorm model (which keeps the written dgrad).
    w = inputs.tiny()
    w.dims = dims
    w.X = inputs.normal_features(w.graph.n, dims[0], 31)
    w.y = inputs.uniform_labels(w.graph.n, dims[-1], 32)
    p0 = _start(variant, dims, 33)
    got, want = util.check_one_step(w, M=3, variant=variant, params0=p0)
    util.check_k_steps_and_average(w, got, want, 3, variant=variant, params0=p0)


def test_variant_flags_are_validated(util, tiny_workload):
    w = tiny_workload
    got = util.gpu_preprocess(w)
    params = util.dev(np.tile(w.params0, (w.M, 1)))
    with pytest.raises(Exception):
        util.ctx().local_steps(w.dims, w.lr, w.M, got["part_host"], got["edge_host"], got["rowptr_out"],
                               got["col_out"], got["Xp"], got["yp"], params, 1, variant=(2, 0, 0))


@pytest.mark.parametrize("variant", [(1, 1, 0), (1, 1, 1)])
def test_variants_with_more_trainers_than_busy_parts(util, variant):
    # 40 nodes over 16 trainers: empty parts, parts of one or two nodes, most nodes isolated
    w = inputs.tiny()
    g = inputs.uniform_graph(40, 100, 3)
    w.graph, w.X, w.y = g, w.X[:40].copy(), w.y[:40].copy()
    p0 = _start(variant, w.dims, 17)
    got, want = util.check_one_step(w, M=16, variant=variant, params0=p0)
    util.check_k_steps_and_average(w, got, want, 2, variant=variant, params0=p0)
