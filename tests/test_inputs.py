"""Host-side checks of the seeded input generators (no GPU)."""
import torch

from paper_2609_33184_b200 import inputs


def test_normal_stream_is_index_addressed_and_gaussian():
    a = inputs.normal_stream(7, inputs.TID_K, 0, 100000)
    b = inputs.normal_stream(7, inputs.TID_K, 5000, 1000)
    assert torch.equal(a[5000:6000], b)
    assert abs(a.mean().item()) < 0.02 and abs(a.std().item() - 1) < 0.02
    assert torch.isfinite(a).all()
    c = inputs.normal_stream(7, inputs.TID_V, 0, 1000)
    assert not torch.equal(a[:1000], c)
    # skew / kurtosis of a normal
    z = (a - a.mean()) / a.std()
    assert abs((z ** 3).mean().item()) < 0.05 and abs((z ** 4).mean().item() - 3) < 0.1


def test_history_is_independent_of_chunking():
    cfg = inputs.scaled(inputs.CONFIGS["c3_internlm25_7b_ragged"], B=2, H_kv=2, H_q=4, d=16,
                        L_c=8, len_lo=13, len_hi=21)
    lens = inputs.history_lengths(cfg)
    assert all(13 <= l <= 21 for l in lens)
    K0, V0, v0 = inputs.make_history_chunk(cfg, 0, lens)
    K1, V1, v1 = inputs.make_history_chunk(cfg, 1, lens)
    assert v0.tolist() == [8, 8] and v1.tolist() == [min(8, l - 8) for l in lens]
    whole = inputs.make_history_block(cfg, inputs.TID_K, 1, 1, 0, lens[1])
    assert torch.equal(whole[:8], K0[1, 1]) and torch.equal(whole[8:8 + v1[1]], K1[1, 1, :v1[1]])
    assert torch.isnan(K1[1, 1, v1[1]:].float()).all() or v1[1] == 8


def test_tree_properties():
    for b in range(4):
        par = inputs.random_tree(inputs.CONFIGS["c4_tree"].seed, b, 64)
        assert len(par) == 64 and par[0] == -1
        depth = [0] * 64
        for i in range(1, 64):
            assert 0 <= par[i] < i
            depth[i] = depth[par[i]] + 1
        assert max(depth) <= 6
        rows = inputs.tree_mask_bits(par)
        for i in range(64):
            m = rows[i][0]
            assert m & 1 and (m >> i) & 1 and m < (1 << (i + 1))
            assert bin(m).count("1") == depth[i] + 1
    assert inputs.random_tree(1, 0, 64) == inputs.random_tree(1, 0, 64)


def test_chain_mask_and_bool_view():
    bits = inputs.mask_bits_tensor([inputs.chain_mask_bits(5)])
    m = inputs.mask_bits_to_bool(bits, 5)[0]
    assert torch.equal(m, torch.tril(torch.ones(5, 5, dtype=torch.bool)))
    bits = inputs.mask_bits_tensor([inputs.tree_mask_bits([-1, 0, 0, 1])])
    m = inputs.mask_bits_to_bool(bits, 4)[0].int().tolist()
    assert m == [[1, 0, 0, 0], [1, 1, 0, 0], [1, 0, 1, 0], [1, 1, 0, 1]]


def test_accept_lengths():
    cfg = inputs.CONFIGS["c5_streamed"]
    idx, cnt = inputs.make_accept(cfg)
    assert idx.shape == (32, 8) and cnt.min() >= 1 and cnt.max() <= 8
    assert len(set(cnt.tolist())) > 3
