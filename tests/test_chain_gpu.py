"""The MLP-stack chain (prune along out -> sparse backward product with f'(z) -> prune along tokens -> sparse
update product, layer after layer) against the same chain run with the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2203_10991_b200 import chain, workloads

pytestmark = pytest.mark.gpu


def to_dev(a):
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


def test_three_layer_chain_matches_oracle_chain():
    T, dims = 512, [256, 384, 128, 256]          # layer i maps dims[i+1] <- dims[i] going up; we walk down
    rng_seed = 5
    layers_np = []
    for i in range(3):                           # top layer first: out = dims[3-i], in = dims[2-i]
        out_f, in_f = dims[3 - i], dims[2 - i]
        layers_np.append({"W": workloads.normal_bf16((out_f, in_f), seed=10 + i, std=in_f ** -0.5),
                          "h": workloads.normal_bf16((T, in_f), seed=20 + i),
                          "act_grad": workloads.normal_bf16((T, in_f), seed=30 + i) if i < 2 else None})
    g_top = workloads.gradient((T, dims[3]), "student_t", seed=rng_seed, dtype="bf16")

    layers_dev = [{k: (None if v is None else to_dev(v)) for k, v in L.items()} for L in layers_np]
    grads = chain.backward_update(to_dev(g_top), layers_dev, base_seed=3)
    torch.cuda.synchronize()

    # oracle chain; the propagated gradient is rounded to bf16 exactly where the GPU chain stores it
    g = g_top
    th = oracle.host_threads()
    for i, L in enumerate(layers_np):
        s_upd, s_bwd = chain.layer_seeds(3, i)
        v, mt = oracle.prune(g, 2, 4, axis=0, seed=s_upd, threads=th)
        want = oracle.gemm(oracle.unpack(v, mt), L["h"], threads=th)
        got = grads[i].double().cpu().numpy()
        err = np.linalg.norm(got - want) / np.linalg.norm(want)
        # layer 0 sees identical inputs; lower layers inherit bf16 roundings of g that may differ by one ulp
        # where the fp32 and fp64 sums straddle a rounding boundary
        assert err <= (2e-5 if i == 0 else 1e-2), (i, err)
        if L["act_grad"] is not None:
            v, mt = oracle.prune(g, 2, 4, axis=1, seed=s_bwd, threads=th)
            dh = oracle.gemm(oracle.unpack(v, mt), L["W"], L["act_grad"], threads=th)
            g = workloads.to_bf16_bits(dh.astype(np.float32))


def test_overlapped_chain_gives_the_same_bits():
    # the two-stream schedule (update product beside the prune that feeds the backward product) runs the same calls
    # with the same seeds: every dW must be bit-identical to the one-stream chain's
    T, dims = 1024, [256, 512, 256, 384]
    layers = []
    for i in range(3):
        out_f, in_f = dims[3 - i], dims[2 - i]
        layers.append({"W": to_dev(workloads.normal_bf16((out_f, in_f), seed=40 + i, std=in_f ** -0.5)),
                       "h": to_dev(workloads.normal_bf16((T, in_f), seed=50 + i)),
                       "act_grad": to_dev(workloads.normal_bf16((T, in_f), seed=60 + i)) if i < 2 else None})
    g_top = to_dev(workloads.gradient((T, dims[3]), "student_t", seed=9, dtype="bf16"))
    for joint in (None, 1):
        a = chain.backward_update(g_top, layers, base_seed=5, joint=joint)
        b = chain.backward_update(g_top, layers, base_seed=5, joint=joint, overlap=True)
        torch.cuda.synchronize()
        for x, y in zip(a, b):
            assert torch.equal(x, y)


def test_chain_with_the_prune_in_the_backward_epilogue_gives_the_same_bits():
    # the backward products prune their own output for the layer below (same seeds, same block numbers): every dW of
    # the chain must be bit-identical to the chain that launches those prunes separately -- alone and with the
    # two-stream schedule; T and the layer widths make both the one-launch route and the two-step route occur
    T, dims = 2048, [256, 2048, 512, 1024]
    layers = []
    for i in range(3):
        out_f, in_f = dims[3 - i], dims[2 - i]
        layers.append({"W": to_dev(workloads.normal_bf16((out_f, in_f), seed=70 + i, std=in_f ** -0.5)),
                       "h": to_dev(workloads.normal_bf16((T, in_f), seed=80 + i)),
                       "act_grad": to_dev(workloads.normal_bf16((T, in_f), seed=90 + i)) if i < 2 else None})
    g_top = to_dev(workloads.gradient((T, dims[3]), "student_t", seed=13, dtype="bf16"))
    for joint in (None, 1):
        a = chain.backward_update(g_top, layers, base_seed=7, joint=joint)
        b = chain.backward_update(g_top, layers, base_seed=7, joint=joint, prune_in_epilogue_min_k=256)
        c = chain.backward_update(g_top, layers, base_seed=7, joint=joint, prune_in_epilogue_min_k=256, overlap=True)
        torch.cuda.synchronize()
        for x, y, z in zip(a, b, c):
            assert torch.equal(x, y) and torch.equal(x, z)
