"""The context's device memory through a caller-supplied allocator (lda_set_allocator): PyTorch's
caching allocator by default in the binding, cudaMalloc on request; the results do not depend on it."""
import numpy as np
import pytest

from paper_1412_1576_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _run(allocator, c):
    g = binding.LightLDA(c.V, c.K, c.alpha, c.beta, allocator=allocator)
    g.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    g.init(5)
    g.sweep(2, 2)
    return g


def test_torch_pool_holds_the_context_and_results_do_not_change():
    import torch
    c = synth.make("small", seed=3)
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    g = _run("torch", c)
    held = torch.cuda.memory_allocated() - before
    st = g.stats()
    assert held >= st["device_bytes"] > 0          # the pool rounds block sizes up, never down
    h = _run("cuda", c)
    assert torch.cuda.memory_allocated() - before == held      # the second context took nothing from the pool
    assert np.array_equal(g.get_assignments(), h.get_assignments())
    assert np.array_equal(g.get_nk(), h.get_nk())
    assert g.loglik() == h.loglik()
    h.close()
    g.close()
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before             # every block went back


def test_allocator_argument_errors():
    c = synth.make("tiny", seed=0)
    g = binding.LightLDA(c.V, c.K, c.alpha, c.beta, allocator="cuda")
    fns = binding.torch_caching_allocator(None)
    assert binding.lda_set_allocator(g._h, fns[0], None) == binding.LDA_EINVAL     # both or neither
    assert binding.lda_set_allocator(g._h, None, None) == 0
    g.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    assert binding.lda_set_allocator(g._h, *fns) == binding.LDA_ESTATE             # only before the corpus is loaded
    g.init(1)
    g.sweep(1, 2)
    with pytest.raises(ValueError):
        binding.LightLDA(c.V, c.K, c.alpha, c.beta, allocator="other")
