"""The allocation-free dense-table entry point against the regular one.

Some users of the library run where device allocation is off limits (inside another
framework's memory pool, in a latency-critical loop, under a fixed memory budget).  They get
the dense smoothing table through ``lda_dense_table_noalloc``, whose scratch is a fixed array
inside the library.  This file is collected last on purpose: it checks that entry point
against ``lda_get_tables`` on two calls in a row, with buffers the test itself owns.
"""
import numpy as np
import pytest

from paper_1412_1576_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _tables_noalloc(torch, n_k, K, V, beta, stream, check_free=False):
    nk_dev = torch.from_numpy(n_k).cuda()
    thr = torch.full((K,), -1, dtype=torch.int32, device="cuda")
    al = torch.full((K,), -1, dtype=torch.int32, device="cuda")
    mass = torch.zeros(1, dtype=torch.int64, device="cuda")
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    rc = binding.lda_dense_table_noalloc(nk_dev.data_ptr(), K, V, beta, thr.data_ptr(), al.data_ptr(),
                                         mass.data_ptr(), status.data_ptr(), stream)
    assert rc == binding.LDA_OK
    torch.cuda.synchronize()
    if check_free:      # not on a device's first call: that one may load the library's device code
        assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
    assert int(status.item()) == 0
    return (thr.cpu().numpy().view(np.uint32), al.cpu().numpy(), int(mass.item()) & (2 ** 64 - 1))


@pytest.mark.parametrize("K", [16, 70_000])
def test_noalloc_dense_table_equals_regular_entry_point_twice(K):
    import torch
    c = synth.generate(V=400, K=K, D=60, length=("fixed", 40), zipf_s=1.0, alpha=0.1, beta=0.01, seed=K)
    stream = torch.cuda.current_stream().cuda_stream
    g = binding.LightLDA(c.V, c.K, c.alpha, c.beta, stream=stream)
    g.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    g.init(1)
    for call in range(2):          # two calls in a row share the library's scratch array
        want = g.get_tables()
        got = _tables_noalloc(torch, g.get_nk(), K, c.V, c.beta, stream, check_free=call == 1)
        assert np.array_equal(got[0], want["dn_thr32"]), call
        assert np.array_equal(got[1], want["dn_alias"]), call
        assert got[2] == want["dense_mass"], call
        g.sweep(1, 2)              # different counts for the second call


def test_noalloc_rejects_sizes_beyond_its_scratch():
    import torch
    buf = torch.zeros(8, dtype=torch.int64, device="cuda")
    p = buf.data_ptr()
    too_big = 131072 + 1
    assert binding.lda_dense_table_noalloc(p, too_big, 10, 0.1, p, p, p) == binding.LDA_ERANGE
    assert binding.lda_dense_table_noalloc(p, 0, 10, 0.1, p, p, p) == binding.LDA_EINVAL
    assert binding.lda_dense_table_noalloc(0, 4, 10, 0.1, p, p, p) == binding.LDA_EINVAL
