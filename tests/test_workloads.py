"""Synthetic layouts: tensor counts and sizes of the five configurations."""
import numpy as np
import torch

from paper_2502_11034_b200 import workloads as W


def test_layout_census():
    tiny = W.build("tiny")
    assert tiny.n_tensors == 8 and tiny.n_params == 528138
    g2 = W.build("gpt2_small")
    assert g2.n_tensors == 148 and g2.n_params == 124439808
    l7 = W.build("llama2_7b")
    assert l7.n_tensors == 9 * 32 + 3 == 291 and l7.n_params == 6738415616
    assert len(l7.extra["spike_tensors"]) == 8
    l1 = W.build("llama32_1b")
    assert l1.n_tensors == 146 and l1.n_params == 1235814400
    ms = W.build("many_small")
    assert ms.n_tensors == 20000 and 1.5e8 < ms.n_params < 2.3e8
    assert min(t.numel for t in ms.tensors) >= 64 and max(t.numel for t in ms.tensors) <= 65536
    moe = W.build("moe_8x1b")
    assert moe.n_tensors == (7 + 3 * 8) * 24 + 3 == 747 and 6.5e9 < moe.n_params < 7.5e9
    assert moe.hyper["beta2"] == 0.999
    ernie = W.build("moe_ernie")                     # the census the paper itself prints: (9 + 3E) L + 3 with E = 48, L = 25
    assert ernie.n_tensors == (9 + 3 * 48) * 25 + 3 == 3828 and 9.5e9 < ernie.n_params < 10.5e9
    for wl in (tiny, g2, l7, l1, ms, moe, ernie):
        offs = np.array([t.offset for t in wl.tensors])
        nums = np.array([t.numel for t in wl.tensors])
        assert (offs % W.ALIGN_ELEMS == 0).all()
        assert (offs[1:] >= offs[:-1] + nums[:-1]).all()
        assert wl.arena_elems >= offs[-1] + nums[-1]


def test_gradient_stream_is_seeded_and_spiked():
    wl = W.build("tiny")
    a, b = W.grads_for_step(wl, 6), W.grads_for_step(wl, 6)
    assert torch.equal(a, b) and a.dtype == torch.float32
    t3 = wl.tensors[3]
    calm = W.grads_for_step(wl, 5)[t3.offset:t3.offset + t3.numel].norm()
    spiked = a[t3.offset:t3.offset + t3.numel].norm()
    assert 50 < float(spiked / calm) < 200
    small = W.build("llama32_1b", n_layer=2, d=64, ffn=128, vocab=512, kv_dim=16)
    g = W.grads_for_step(small, 1)
    assert g.dtype == torch.bfloat16 and g.numel() == small.arena_elems
    k = max(1, round(0.05 * small.n_tensors))
    assert len(W.spikes_for_step(small, 3)) == k
    assert W.spikes_for_step(small, 3) == W.spikes_for_step(small, 3)
    mini = W.build("many_small", n_tensors=50)
    gm = W.grads_for_step(mini, 2)
    last = mini.tensors[-1]
    assert float(gm[last.offset + last.numel:].abs().sum()) == 0.0
