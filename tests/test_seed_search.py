"""Exhaustive seed search (Section 5.2): the host path that builds a blob from given seeds (CPU)
and the GPU search against the oracle's exhaustive encoder, bit for bit."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_1905_10138_b200 import sqnn
from paper_1905_10138_b200 import workloads as wl
from tests import helpers as H
from tests.test_gpu_decode import generic_layer


def packed(layer):
    return (np.concatenate([wl.pack_bits(layer.planes[i]) for i in range(layer.n_q)]), wl.pack_bits(layer.mask))


def test_blob_from_given_seeds_matches_exhaustive_encoder_and_any_seed_is_lossless():
    layer = wl.make_layer(1, m=40, n=100)
    planes_words, mask_words = packed(layer)
    rows = wl.network_rows(layer.M)
    ref_blob, ref_stats = H.blob_from_library(layer, sqnn.ENCODE_EXHAUSTIVE)
    owc, onp, odp = orc.encode_plane(layer.M, layer.planes[0].ravel(), layer.mask.ravel(), exhaustive=True)
    blob, stats = sqnn.sqnn_encode_seeds_host(rows, layer.n_in, layer.m, layer.n, 1, planes_words, mask_words,
                                              [owc.astype(np.uint32)])
    assert np.array_equal(blob, ref_blob) and stats["patches"] == ref_stats["patches"]
    # arbitrary seeds still give a lossless blob (more patches)
    rng = np.random.default_rng(3)
    junk = rng.integers(0, 1 << layer.n_in, owc.size, dtype=np.uint32)
    blob2, stats2 = sqnn.sqnn_encode_seeds_host(rows, layer.n_in, layer.m, layer.n, 1, planes_words, mask_words, [junk])
    wc, np_, dp = sqnn.sqnn_unpack_host(blob2, 0)
    out = orc.decode_plane(layer.M, layer.mn, wc.astype(np.uint64), np_, dp)
    care = layer.mask.ravel() == 1
    assert np.array_equal(out[care], layer.planes[0].ravel()[care])
    assert stats2["patches"][0] >= stats["patches"][0]
    with pytest.raises(sqnn.SqnnError) as e:
        bad = junk.copy()
        bad[0] = 1 << layer.n_in
        sqnn.sqnn_encode_seeds_host(rows, layer.n_in, layer.m, layer.n, 1, planes_words, mask_words, [bad])
    assert e.value.status == sqnn.E_INVALID_ARG


SEARCH = [
    ("80x8", lambda: wl.make_layer(1, m=64, n=250)),
    ("100x10", lambda: wl.make_layer(2, m=12, n=1000)),
    ("60x12-q2", lambda: wl.make_layer(3, m=10, n=300)),
    ("13x5", lambda: generic_layer(13, 5, 17, 101, 0.5, 31)),
    ("8x3", lambda: generic_layer(8, 3, 9, 77, 0.6, 32)),
    ("200x10", lambda: generic_layer(200, 10, 11, 1000, 0.1, 33)),
    ("40x14", lambda: generic_layer(40, 14, 5, 333, 0.4, 34)),
]


@pytest.mark.gpu
@pytest.mark.parametrize("name,make", SEARCH, ids=[s[0] for s in SEARCH])
def test_gpu_seed_search_matches_oracle_exhaustive(name, make):
    import torch
    layer = make()
    planes_words, mask_words = packed(layer)
    rows = wl.network_rows(layer.M)
    l = (layer.mn + layer.n_out - 1) // layer.n_out
    d_planes = torch.from_numpy(planes_words.view(np.int64)).cuda()
    d_mask = torch.from_numpy(mask_words.view(np.int64)).cuda()
    d_wc = torch.full((layer.n_q * l,), -1, dtype=torch.int32, device="cuda")
    d_np = torch.full((layer.n_q * l,), -1, dtype=torch.int16, device="cuda")
    sqnn.sqnn_search_seeds(rows, layer.n_in, layer.m, layer.n, layer.n_q, d_planes, d_mask, d_wc, d_np)
    torch.cuda.synchronize()
    wc = d_wc.cpu().numpy().view(np.uint32).reshape(layer.n_q, l)
    np_ = d_np.cpu().numpy().view(np.uint16).reshape(layer.n_q, l)
    care = layer.mask.ravel()
    for i in range(layer.n_q):
        owc, onp, odp = orc.encode_plane(layer.M, layer.planes[i].ravel(), care, exhaustive=True)
        assert np.array_equal(wc[i].astype(np.uint64), owc), (name, i)
        assert np.array_equal(np_[i], onp)
    # the blob built from these seeds decodes to every care bit and needs no more patches than Algorithm 1
    blob, stats = sqnn.sqnn_encode_seeds_host(rows, layer.n_in, layer.m, layer.n, layer.n_q, planes_words, mask_words,
                                              [wc[i] for i in range(layer.n_q)])
    _, stats_a = H.blob_from_library(layer)
    dev = H.DeviceLayer(layer, blob)
    got = dev.decode_bits()
    for i in range(layer.n_q):
        bits = wl.unpack_bits(got[i], layer.mn)
        assert np.array_equal(bits[care == 1], layer.planes[i].ravel()[care == 1])
        assert stats["patches"][i] == int(np_[i].sum()) <= stats_a["patches"][i]
