"""GPU parity of the group construction (pcg_asg_create) against the CPU oracle: the CSR must be identical
(group_ptr, group_tok, tok_degree are integer outputs), on tables whose every pair decision is further from the
threshold than the float32 rounding of the kernel's cosine (the oracle reports the smallest margin)."""
import numpy as np
import pytest

from paper_2511_13732_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

BAND = 2e-5  # |cos - theta| below this may legitimately flip between float64 and the kernel's float32 cosine


def _to_device(emb):
    if emb.dtype == np.uint16:
        return torch.from_numpy(emb.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(emb).cuda()


def _clear_threshold(emb, theta0, width=0.02):
    """A threshold near theta0 that no pair's cosine comes closer to than 5 bands (middle of the largest gap)."""
    from oracle import asg_oracle as A

    E = A.widen(emb)
    n = np.sqrt((E * E).sum(1))
    cos = (E @ E.T) / np.maximum(n[:, None] * n[None, :], 1e-300)
    c = np.sort(cos[np.triu_indices(E.shape[0], 1)])
    c = c[(c > theta0 - width) & (c < theta0 + width)]
    c = np.concatenate([[theta0 - width], c, [theta0 + width]])
    k = int(np.argmax(np.diff(c)))
    assert c[k + 1] - c[k] > 10 * BAND
    return float(np.float32(0.5 * (c[k] + c[k + 1])))


def _check(emb, theta):
    """Both tensor-core paths (tcgen05 and mma.sync) against the oracle."""
    from oracle import asg_oracle as A
    from paper_2511_13732_b200 import binding

    want = A.build_groups(emb, theta)
    assert want.min_margin > BAND, "test table has a pair too close to the threshold"
    for mma_sync in (False, True):
        asg = binding.Asg(_to_device(emb), theta, mma_sync=mma_sync)
        assert asg.info.tensor_path == (0 if mma_sync else 1)
        gp, gt, dg = asg.csr_arrays()
        assert asg.info.M == want.M and asg.info.nnz == want.group_tok.size
        assert np.array_equal(gp, want.group_ptr) and np.array_equal(gt, want.group_tok)
        assert np.array_equal(dg, want.tok_degree)
        sizes = np.diff(want.group_ptr)
        assert asg.info.max_group_size == sizes.max() and asg.info.max_degree == want.tok_degree.max()
    return asg, want


def _clustered(rng, V, d, centres, noise=0.05, bridges=0):
    c = rng.standard_normal((centres, d)).astype(np.float32)
    c /= np.linalg.norm(c, axis=1, keepdims=True)
    which = rng.integers(0, centres, V)
    emb = c[which] * rng.uniform(0.5, 2.0, (V, 1)).astype(np.float32) + noise * rng.standard_normal((V, d)).astype(np.float32) / np.sqrt(d)
    for t in rng.choice(V, bridges, replace=False):  # tokens half-way between two clusters: overlapping groups
        a, b = rng.choice(centres, 2, replace=False)
        emb[t] = c[a] + c[b]
    return emb.astype(np.float32)


@pytest.mark.parametrize("V,d,dtype", [(3000, 48, "bf16"), (1000, 100, "f32"), (130, 7, "bf16"), (4096, 64, "bf16")])
def test_clustered_tables_with_duplicates_and_overlaps(V, d, dtype):
    rng = np.random.default_rng(V + d)
    emb = _clustered(rng, V, d, centres=40, bridges=V // 20)
    emb[7] = 0.0  # a zero embedding: similar to nothing but itself
    emb[11] = 2.0 * emb[5]  # exact duplicate direction: identical neighbourhoods
    if dtype == "bf16":
        emb = W.f32_to_bf16_bits(emb)
    theta = _clear_threshold(emb, 0.6)
    asg, want = _check(emb, theta)
    assert want.M < V  # identical neighbourhoods were merged
    assert want.tok_degree.max() > 1  # and groups overlap


def test_random_table_near_the_papers_threshold():
    rng = np.random.default_rng(5)
    emb = W.f32_to_bf16_bits(rng.standard_normal((520, 32)).astype(np.float32))
    theta = _clear_threshold(emb, 0.42, width=0.03)  # the paper finds thresholds of 0.38-0.45 best
    _check(emb, theta)


def test_limiting_thresholds():
    rng = np.random.default_rng(6)
    emb = rng.standard_normal((300, 16)).astype(np.float32)
    asg, want = _check(emb, -1.5)
    assert asg.info.M == 1 and asg.info.max_group_size == 300
    asg, want = _check(emb, 1.5)
    assert asg.info.M == 300 and asg.info.nnz == 300


def test_constructed_groups_feed_verification(oracle):
    """End to end: groups built on the GPU go straight into pcg_groups_create and pcg_verify, and the result equals
    the oracle's verification on the oracle's groups."""
    from oracle import asg_oracle as A
    from oracle.compare import compare_verify
    from paper_2511_13732_b200 import binding

    from gpu_util import logits_to_device

    rng = np.random.default_rng(8)
    V, B, K = 1500, 12, 4
    emb = W.f32_to_bf16_bits(_clustered(rng, V, 24, centres=60, bridges=100))
    theta = _clear_threshold(emb, 0.6, width=0.08)
    want = A.build_groups(emb, theta)
    handle = binding.Asg(_to_device(emb), theta).groups()
    assert handle.M == want.M
    tl = (2.0 * rng.standard_normal((B, K + 1, V))).astype(np.float32)
    dl = (tl[:, :K] + 0.7 * rng.standard_normal((B, K, V))).astype(np.float32)
    x = np.argmax(dl + rng.gumbel(size=dl.shape), axis=2).astype(np.int32)
    u = (rng.integers(0, 1 << 24, (B, K + 1, 2)) * 2.0 ** -24).astype(np.float32)
    ref = oracle.verify(tl, dl, x, want.group_ptr, want.group_tok, want.tok_degree, u, 1.0, threads=0)
    n, tok, grp, flg = binding.pcg_verify(logits_to_device(tl), logits_to_device(dl), torch.from_numpy(x).cuda(), handle,
                                          torch.from_numpy(u).cuda(), 1.0)
    cmp = compare_verify(n.cpu().numpy(), tok.cpu().numpy(), grp.cpu().numpy(), ref)
    assert cmp.hard == 0 and cmp.excused == 0, cmp.details[:3]


def test_argument_errors():
    from paper_2511_13732_b200 import binding

    emb = torch.zeros((4, 4), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.PcgError) as err:
        binding.Asg(emb, float("nan"))
    assert err.value.status == 1


def _clear_threshold_chunked(emb, lo, hi, chunk=1024):
    """As _clear_threshold for tables too large to hold all cosines: only those inside (lo, hi) are collected."""
    from oracle import asg_oracle as A

    E = A.widen(emb)
    n = np.sqrt((E * E).sum(1))
    En = E / np.maximum(n, 1e-300)[:, None]
    near = [np.array([lo, hi])]
    for r0 in range(0, E.shape[0], chunk):
        cos = En[r0:r0 + chunk] @ En.T
        near.append(cos[(cos > lo) & (cos < hi)])
    c = np.sort(np.concatenate(near))
    k = int(np.argmax(np.diff(c)))
    assert c[k + 1] - c[k] > 10 * BAND
    return float(np.float32(0.5 * (c[k] + c[k + 1])))


def test_large_table_of_sixteen_thousand_tokens():
    """V = 16,384 (128 x 64 tiles of the tensor-core kernel, several waves of its persistent blocks), both tensor
    paths: clusters with duplicated rows and bridge tokens, the threshold in the widest gap of the cosines near 0.6."""
    rng = np.random.default_rng(16)
    emb = _clustered(rng, 16384, 96, 700, noise=0.03, bridges=300)
    emb[5000:5040] = emb[100:140]  # duplicated embeddings: identical neighbourhoods must merge
    asg, want = _check(emb, _clear_threshold_chunked(emb, 0.58, 0.62))
    assert want.M < 16384 and want.tok_degree.max() >= 2
