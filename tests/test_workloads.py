"""The seeded input generators: draw order, shapes and page structure of the synthetic configs."""
import numpy as np
import pytest
import torch

import wpp_workloads as W


def test_counter_stream_is_sliceable_and_deterministic():
    a = W.counter_normal_bf16(7, 2, 0, 5000)
    b = W.counter_normal_bf16(7, 2, 1234, 100)
    assert torch.equal(a[1234:1334], b)
    assert not torch.equal(W.counter_normal_bf16(7, 3, 0, 100), a[:100])
    assert not torch.equal(W.counter_normal_bf16(8, 2, 0, 100), a[:100])


def test_counter_stream_looks_standard_normal():
    x = W.counter_normal_bf16(1, 0, 0, 1 << 20).double()
    assert abs(x.mean().item()) < 5e-3 and abs(x.std().item() - 1) < 5e-3
    assert 3.5 < x.abs().max().item() < 4.5 and torch.isfinite(x).all()


def test_cfg1_shape():
    w = W.cfg1()
    assert (w.num_requests, w.total_new_tokens, w.head_dim, w.page_size) == (1, 128, 64, 16)
    assert (w.num_q_heads, w.num_kv_heads) == (8, 2) and w.unique_kv_pages() == 24
    assert w.flops == 4 * 64 * 8 * (128 * 256 + 128 * 129 // 2)


def test_cfg2_lengths():
    w = W.cfg2()
    assert w.num_requests == 16 and np.all(w.prefix_lens % 64 == 0)
    assert w.prefix_lens.max() <= 8192 and 256 <= w.chunk_lens.min() and w.chunk_lens.max() <= 2048
    assert w.total_new_tokens == 17933


def test_cfg3_sharing_structure():
    w = W.cfg3()
    assert w.num_requests == 128 and w.total_new_tokens == 278426
    sharers = w.prefix_lens >= 16384
    assert sharers.sum() == 102
    first = w.block_tables[np.argmax(sharers), :256]
    for i in np.nonzero(sharers)[0]:
        assert np.array_equal(w.block_tables[i, :256], first)
    # every non-shared page is referenced by exactly one table
    ids, counts = np.unique(w.block_tables[w.block_tables >= 0], return_counts=True)
    assert set(ids[counts > 1]) == set(first.tolist()) and ids.size == 9285
    # most private suffixes start in the middle of a page
    assert (w.prefix_lens % 64 != 0).sum() > 100


def test_cfg4_scale_exponents():
    w = W.cfg4(num_requests=2, prefix=3 * 4096, chunk=4096 + 64)
    assert w.page_scale_log2.max() == 4 and w.token_scale_log2[0] == 3 and w.token_scale_log2[4096] == 4
    for i in range(2):
        assert np.array_equal(w.page_scale_log2[w.block_tables[i, :256]], np.repeat(np.arange(4), 64))
    wa = W.cfg4("alternate", num_requests=1, prefix=3 * 4096, chunk=64)
    assert set(np.unique(wa.page_scale_log2)) == {0, 1}
    k = w.k_pool(start_page=int(w.block_tables[0, 64]), pages=1).double()
    assert k.abs().max() > 4.4          # scaled by 2


def test_block_tables_are_disjoint_without_sharing():
    w = W.custom_workload([5, 0, 130], [9, 70, 1], 4, 2, 8, 16, seed=3)
    ids = w.block_tables[w.block_tables >= 0]
    assert np.unique(ids).size == ids.size and ids.max() < w.num_pages
    need = (w.prefix_lens + w.chunk_lens + 15) // 16
    assert [(r >= 0).sum() for r in w.block_tables] == need.tolist()


@pytest.mark.gpu
def test_counter_stream_is_identical_on_cpu_and_gpu():
    a = W.counter_normal_bf16(5, 1, 77, 1 << 18, device="cpu")
    b = W.counter_normal_bf16(5, 1, 77, 1 << 18, device="cuda")
    assert torch.equal(a, b.cpu())
