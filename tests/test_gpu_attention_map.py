"""The cast of the attention map inside the fused attention kernel (the path full-size attention runs): the
kernel's own bf16 map, fed to the oracle quantizer, must give the kernel's codes and scales bit for bit; the
positive plane it feeds to the tensor cores must equal the codes, its UE4M3 scale factors a host-side conversion
of the oracle's scales, and no scale may be flushed.  The map itself is checked against the all-CPU pipeline
(fp32 exp on the device against fp64 on the host: single bf16 roundings differ), and the output O - computed by
the same kernel from the map it never stores - against the oracle's product of the kernel's own quantized map
with the quantized V."""
import numpy as np
import pytest
import torch

import oracle
from paper_2411_09909_b200 import amx, inputs

pytestmark = pytest.mark.gpu


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def e5m2_key_mant(b):
    """E5M2 byte -> (exponent key = unbiased exponent + 17, two mantissa bits) of its normalised form; key 0 = zero."""
    b = b.astype(np.int64)
    key = np.where(b >= 4, (b + 8) >> 2, np.array([0, 1, 2, 2])[np.minimum(b, 3)])
    mant = np.where(b >= 4, b & 3, np.array([0, 0, 0, 2])[np.minimum(b, 3)])
    return key, mant


def expected_scale_factors(scale_pos, kmax):
    """UE4M3 bytes of the positive-side scales [rows, G] under the per-row offset (largest key kmax [rows])."""
    key, mant = e5m2_key_mant(scale_pos)
    field = key - kmax[:, None] + 15
    return np.where((scale_pos != 0) & (field >= 1), (field << 3) | (mant << 1), 0).astype(np.uint8)


def check_rows(rows, L, p_bits, codes, scales, prep, causal):
    """rows: row indices to check.  p_bits/codes/scales: host arrays of the whole map."""
    oc, os_ = oracle.quantize(np.ascontiguousarray(p_bits[rows]), 32)
    assert np.array_equal(codes[rows], oc)
    assert np.array_equal(scales[rows], os_)
    assert not np.any(os_[:, :, 1])                                  # no negative side in a softmax output
    plane_bytes = -(-(L * L // 2) // 256) * 256
    nk64 = -(-L // 256) * 4
    sf_bytes = (L // 128) * nk64 * 512
    plane = prep[: L * L // 2].reshape(L, L // 2)
    G = L // 32
    if causal:          # blocks of 128 keys entirely after the query's block of 128 are never visited nor read
        for i, r in enumerate(rows):
            seen = (r // 128 + 1) * 128 // 2
            assert np.array_equal(plane[r, :seen], oc[i, :seen])
    else:
        assert np.array_equal(plane[rows], oc)
    sf = prep[2 * plane_bytes: 2 * plane_bytes + sf_bytes]
    words = prep[2 * plane_bytes + 2 * sf_bytes: 2 * plane_bytes + 2 * sf_bytes + 4 * L].view(np.int32)
    key, _ = e5m2_key_mant(os_[:, :, 0])
    kmax = key.max(axis=1)
    assert np.array_equal((words[rows] & 0xFFFF).astype(np.int16).astype(np.int64), kmax - 25)
    assert np.all((words[rows] >> 16) & 3 == 1) and np.all(words[rows] >> 18 == 0)   # positive side only, nothing flushed
    want = expected_scale_factors(os_[:, :, 0], kmax)
    for i, r in enumerate(rows):
        g = np.arange(G if not causal else (r // 128 + 1) * 4)
        off = (r // 128) * nk64 * 512 + (g // 2) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + (g % 2) * 2
        assert np.array_equal(sf[off], want[i, g]) and np.array_equal(sf[off + 1], want[i, g]), r


def check_output(o, rows, codes, scales, vb):
    """O of the sampled rows against the oracle's product of the kernel's own quantized map with the quantized V."""
    vq = oracle.quantize(np.ascontiguousarray(vb.T), 32)
    ref = oracle.gemm(np.ascontiguousarray(codes[rows]), np.ascontiguousarray(scales[rows]), *vq, 32)
    got = o[rows].astype(np.float64)
    assert np.linalg.norm(got - ref) <= 1e-5 * np.linalg.norm(ref)


@pytest.mark.parametrize("L", [128, 384, 512])
@pytest.mark.parametrize("causal", [False, True])
def test_attention_map_cast_bit_exact_small(L, causal):
    qb, kb, vb = (t[0] for t in inputs.attention_qkv(heads=1, seq=L))
    flags = amx.ATTN_CAUSAL if causal else 0
    o, p, c, s, prep = amx.attention_map(dev_bf16(qb), dev_bf16(kb), dev_bf16(vb), flags)
    p_bits = p.view(torch.int16).cpu().numpy().view(np.uint16)
    check_rows(np.arange(L), L, p_bits, c.cpu().numpy(), s.cpu().numpy(), prep.cpu().numpy(), causal)
    check_output(o.cpu().numpy(), np.arange(L), c.cpu().numpy(), s.cpu().numpy(), vb)
    assert amx.prepared_flushed_scales(prep, L, L, False) == 0
    # amx_attention gives the same output for the head (same kernels)
    heads = amx.attention_heads(dev_bf16(qb)[None], dev_bf16(kb)[None], dev_bf16(vb)[None], flags=flags | amx.GEMM_FP4)
    assert torch.equal(heads[0], o)
    # the map itself against the all-CPU pipeline: equal up to one bf16 ulp on a small share of the entries
    S = oracle.gemm(*oracle.quantize(qb, 32), *oracle.quantize(kb, 32), 32)
    want = oracle.softmax_bf16(S, 128 ** -0.5, causal_row0=0) if causal else oracle.softmax_bf16(S, 128 ** -0.5)
    diff = np.abs(p_bits.astype(np.int32) - want.astype(np.int32))
    assert diff.max() <= 1 and np.mean(diff != 0) < 0.02
    if causal:
        assert not np.any(np.triu(p_bits, 1))                        # masked entries are exactly +0


def test_attention_map_softer_rows_bit_exact():
    """Inputs scaled down so that rows of the map hold many nonzero groups of very different size (the benchmark's
    inputs make it nearly one-hot): exercises the scale-factor range of the cast."""
    L = 512
    qb, kb, vb = (t[0] for t in inputs.attention_qkv(heads=1, seq=L))
    small = lambda b: inputs.f32_to_bf16_bits(inputs.bf16_bits_to_f32(b) * 0.35)
    qb, kb = small(qb), small(kb)
    o, p, c, s, prep = amx.attention_map(dev_bf16(qb), dev_bf16(kb), dev_bf16(vb), 0)
    p_bits = p.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.mean(s.cpu().numpy()[:, :, 0] != 0) > 0.5
    check_rows(np.arange(L), L, p_bits, c.cpu().numpy(), s.cpu().numpy(), prep.cpu().numpy(), False)
    check_output(o.cpu().numpy(), np.arange(L), c.cpu().numpy(), s.cpu().numpy(), vb)


@pytest.mark.parametrize("causal", [False, True])
def test_attention_map_cast_bit_exact_full_size_sampled(causal):
    """Config-5 size (8192 keys): three sampled blocks of 128 query rows of head 0."""
    L = 8192
    qb, kb, vb = (t[0] for t in inputs.attention_qkv(heads=1, seq=L))
    flags = amx.ATTN_CAUSAL if causal else 0
    o, p, c, s, prep = amx.attention_map(dev_bf16(qb), dev_bf16(kb), dev_bf16(vb), flags)
    p_bits = p.view(torch.int16).cpu().numpy().view(np.uint16)
    rng = np.random.default_rng(77)
    blocks = np.sort(rng.choice(L // 128, size=3, replace=False))
    rows = np.concatenate([np.arange(b * 128, b * 128 + 128) for b in blocks])
    c_np, s_np = c.cpu().numpy(), s.cpu().numpy()
    check_rows(rows, L, p_bits, c_np, s_np, prep.cpu().numpy(), causal)
    check_output(o.cpu().numpy(), rows[::4], c_np, s_np, vb)
    assert amx.prepared_flushed_scales(prep, L, L, False) == 0


@pytest.mark.parametrize("heads,kv_heads,L,d,flags", [(8, 2, 256, 128, amx.GEMM_FP4),                    # fused kernel, groups of 4
                                                       (20, 4, 128, 128, amx.GEMM_FP4 | amx.ATTN_CAUSAL),  # groups of 5: chunks of 15 heads
                                                       (34, 1, 128, 128, amx.GEMM_FP4),                    # one group larger than a chunk
                                                       (6, 2, 160, 64, amx.GEMM_AUTO),                     # stored logits, head by head
                                                       (9, 3, 256, 128, amx.GEMM_TC | amx.ATTN_CAUSAL)])   # chunks of 8 heads, groups of 3
def test_grouped_query_attention_equals_repeated_heads(heads, kv_heads, L, d, flags):
    """amx_attention_gqa: query head h uses head h / (heads / kv_heads) of keys and values - the same bits as
    amx_attention on keys and values repeated; one head also against the all-CPU pipeline."""
    rng = np.random.default_rng(heads * 100 + kv_heads)
    def bf(shape):
        return torch.from_numpy(inputs.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32)).view(np.int16)).cuda().view(torch.bfloat16)
    q, k, v = bf((heads, L, d)), bf((kv_heads, L, d)), bf((kv_heads, L, d))
    g = heads // kv_heads
    got = amx.attention_heads(q, k, v, flags=flags)
    want = amx.attention_heads(q, k.repeat_interleave(g, dim=0).contiguous(), v.repeat_interleave(g, dim=0).contiguous(), flags=flags)
    assert torch.equal(got, want)
    h = heads - 1
    u16 = lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)
    qb, kb, vb = u16(q[h]), u16(k[h // g]), u16(v[h // g])
    S = oracle.gemm(*oracle.quantize(qb, 32), *oracle.quantize(kb, 32), 32)
    P = oracle.softmax_bf16(S, d ** -0.5, causal_row0=0) if flags & amx.ATTN_CAUSAL else oracle.softmax_bf16(S, d ** -0.5)
    ref = oracle.gemm(*oracle.quantize(P, 32), *oracle.quantize(np.ascontiguousarray(vb.T), 32), 32).astype(np.float64)
    assert np.linalg.norm(got[h].cpu().numpy() - ref) <= 1e-3 * np.linalg.norm(ref)
    L_ = amx.lib()
    assert L_.amx_attention_gqa(q.data_ptr(), k.data_ptr(), v.data_ptr(), heads, heads + 1, L, d, 0, got.data_ptr(), None, 0, None) == -2
