"""GPU parity: INT8-KV decode attention against the CPU oracle's tiled mode (which mirrors the kernel's tile and
split schedule), within 1e-3 of the row L2 norm; plus the accuracy ordering against the dequantize-to-BF16 path."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_13915_b200 import binding, inputs
from helpers import bf16_dev, bf16_bits, dev, rel_row_err

pytestmark = pytest.mark.gpu
TOL = 1e-3


def _split_starts(c, all_seqlens=None, max_seqlen=None, q_len=1, paged=False):
    """The kernel's context splits for every (sequence, query head) of a call over sequences of these lengths:
    ([B, Hkv, q_len * Hq / Hkv, n_splits + 1] token offsets, tile)."""
    Hq, D = c.q.shape[1] // q_len, c.q.shape[2]
    L = np.diff(c.cu_seqlens) if all_seqlens is None else np.asarray(all_seqlens)
    return binding.attn_decode_split_starts(L, Hq, c.k.shape[1], D, c.dv, max(max_seqlen or int(L.max()), 1), q_len=q_len,
                                            paged=paged, v_aliased=c.v is None)


def _run_gpu(c, want_lse=True):
    B, Hq, D = c.q.shape
    Hkv = c.k.shape[1]
    q = bf16_dev(c.q)
    k = dev(c.k)
    v = None if c.v is None else dev(c.v)
    ks = dev(c.k_scale)
    vs = None if c.v_scale is None else dev(c.v_scale)
    cu = dev(c.cu_seqlens)
    out = binding.attn_decode_int8kv(q, k, v, ks, vs, cu, max(c.max_seqlen, 1), c.softmax_scale, dv=c.dv, want_lse=want_lse)
    torch.cuda.synchronize()
    binding.last_device_status()
    return out


def _oracle_tiled(c, all_seqlens=None, seqs=None, max_seqlen=None, paged=False):
    """The oracle's tiled mode on case c with the splits the kernel takes.  all_seqlens / seqs: c holds only the
    sequences `seqs` of a call over sequences of lengths all_seqlens (the splits depend on all of them)."""
    B, Hq, D = c.q.shape
    Hkv = c.k.shape[1]
    starts, tile = _split_starts(c, all_seqlens, max_seqlen, paged=paged)
    ss = starts.reshape(starts.shape[0], Hq, -1)
    if seqs is not None:
        ss = ss[seqs]
    shape = (starts.shape[0], Hq, Hkv, D, c.dv, max(max_seqlen or c.max_seqlen, 1))
    return oracle.attn_decode_int8kv(c.q, c.k, c.v, c.k_scale, c.v_scale, c.cu_seqlens, c.softmax_scale, dv=c.dv,
                                     split_starts=np.ascontiguousarray(ss), tile=tile, want_lse=True, **_softmax_mode(*shape))


def _softmax_mode(*shape):
    """Which tiled mode of the oracle mirrors the kernel for this shape: the plain online softmax, or the one whose
    references are held between tiles (wide head groups), with the margins the library reports."""
    margin, growth = binding.attn_decode_softmax_rule(*shape)
    if growth == 0.0:
        return dict(mode="tiled")
    return dict(mode="held", m_margin=margin, sv_growth=growth)


def _assert_close(got, ref):
    """|y - y_oracle| <= 1e-3 * ||y_oracle row||_2 for the FP32 result, plus the final rounding to BF16 that both the
    kernel and a BF16 consumer of the oracle's value incur (one BF16 ulp = 2^-8 relative at most)."""
    n = np.linalg.norm(ref, axis=-1, keepdims=True)
    assert np.all(np.abs(got - ref) <= TOL * n + np.abs(ref) * 2.0 ** -8 + 1e-30), \
        float((np.abs(got - ref) - np.abs(ref) * 2.0 ** -8).max() / n.max())


def _check(c):
    o, lse = _run_gpu(c)
    ref, lse_ref = _oracle_tiled(c)
    got = oracle.bf16_bits_to_f64(bf16_bits(o))
    _assert_close(got, ref)
    live = np.isfinite(lse_ref)
    assert np.allclose(lse.cpu().numpy()[live], lse_ref[live], rtol=0, atol=2e-3)
    assert np.all(np.isneginf(lse.cpu().numpy()[~live]))
    return got, ref


@pytest.mark.parametrize("B,Hq,Hkv,seqlens", [
    (1, 4, 1, [128]), (3, 8, 2, [700, 64, 1500]), (2, 32, 8, [129, 4000]), (4, 8, 8, [1, 127, 0, 300]),
    (2, 32, 2, [513, 2222]), (1, 24, 2, [999]),
])
def test_gqa_parity(B, Hq, Hkv, seqlens):
    _check(inputs.gqa_case(B, Hq, Hkv, 128, seqlens, seed=B + Hq))


@pytest.mark.parametrize("seqlens", [[300, 1000], [16384 // 8]])
def test_mla_parity(seqlens):
    _check(inputs.mla_case(len(seqlens), 64, 576, 512, seqlens, seed=11))


def test_other_head_dims():
    c = inputs.gqa_case(2, 8, 2, 64, [400, 77], seed=5)          # D = Dv = 64: half-filled chunk
    _check(c)
    c = inputs.gqa_case(2, 4, 2, 256, [300, 640], seed=6)        # two chunks of D and Dv
    _check(c)


@pytest.mark.parametrize("splits", ["1", "2", "7"])
def test_split_counts(splits, monkeypatch):
    binding.debug_set_option("MSD_ATTN_SPLITS", int(splits))
    _check(inputs.gqa_case(2, 8, 2, 128, [1000, 3000], seed=9))


# ---- the balanced split schedule (equal runs of the list of all sequences' tiles, one CTA per run and unit) ------------
@pytest.mark.parametrize("B,Hq,Hkv,seqlens", [
    (3, 8, 2, [700, 64, 1500]),                       # runs that cross sequence boundaries
    (4, 8, 8, [1, 127, 0, 300]),                      # one row per KV head, an empty sequence in the middle
    (2, 32, 8, [129, 4000]),                          # many runs inside one sequence
    (6, 12, 4, [0, 0, 513, 0, 90, 0]),                # empty sequences first, between and last; 3 rows per KV head
    (1, 4, 1, [128]),                                 # a single tile
    (3, 16, 2, [700, 64, 1500]),                      # 8 rows per KV head
    (2, 14, 2, [0, 2100]),                            # 7 rows per KV head
])
def test_balanced_schedule_parity(B, Hq, Hkv, seqlens):
    binding.debug_set_option("MSD_ATTN_BALANCED", 1)
    c = inputs.gqa_case(B, Hq, Hkv, 128, seqlens, seed=3 * B + Hq)
    assert binding.attn_decode_schedule(B, Hq, Hkv, 128, 128, max(c.max_seqlen, 1))[2] == 0      # the balanced schedule is in force
    _check(c)


def test_balanced_schedule_many_short_sequences():
    """Every CTA walks several sequences (segments), some of them empty, with a different number of tiles each."""
    binding.debug_set_option("MSD_ATTN_BALANCED", 1)
    rng = np.random.default_rng(5)
    seqlens = [int(x) for x in rng.integers(0, 1200, 300)]
    seqlens[7] = seqlens[8] = seqlens[299] = 0
    c = inputs.gqa_case(len(seqlens), 8, 2, 128, seqlens, seed=77)
    starts, _ = _split_starts(c)
    assert (np.diff(starts[:, 0, 0], axis=1) > 0).sum(axis=1).max() >= 2       # some sequence is cut by a run boundary
    _check(c)


def test_balanced_schedule_is_the_default_where_it_pays():
    """Between one and three fixed splits per resident CTA the balanced schedule is taken; with many more it is not."""
    assert binding.attn_decode_schedule(32, 32, 8, 128, 128, 8192)[2] == 0
    assert binding.attn_decode_schedule(512, 32, 8, 128, 128, 8192)[2] > 0
    assert binding.attn_decode_schedule(1, 32, 8, 128, 128, 8192)[2] > 0
    assert binding.attn_decode_schedule(32, 64, 8, 128, 128, 8192)[2] == 0       # 8 rows per KV head as well
    assert binding.attn_decode_schedule(32, 128, 8, 128, 128, 8192)[2] > 0       # 16 rows per KV head: fixed splits
    assert binding.attn_decode_schedule(256, 32, 8, 128, 128, 1024)[2] > 0       # short sequences: fixed splits
    binding.debug_set_option("MSD_ATTN_BALANCED", 0)
    assert binding.attn_decode_schedule(32, 32, 8, 128, 128, 8192)[2] > 0


def test_balanced_schedule_sequence_longer_than_declared():
    """A sequence longer than the max_seqlen the workspace was sized for: reported, nothing written out of bounds
    (the guard bands of the workspace are checked when the test ends)."""
    binding.debug_set_option("MSD_ATTN_BALANCED", 1)
    c = inputs.gqa_case(1, 8, 2, 128, [4000], seed=4)
    binding.attn_decode_int8kv(bf16_dev(c.q), dev(c.k), dev(c.v), dev(c.k_scale), dev(c.v_scale), dev(c.cu_seqlens), 512,
                               c.softmax_scale, dv=c.dv)
    torch.cuda.synchronize()
    with pytest.raises(binding.MsdError) as e:
        binding.last_device_status()
    assert e.value.code == 2                          # MSD_ERR_BAD_SHAPE
    binding.last_device_status()                      # cleared


def test_accuracy_ordering_vs_dequant():
    c = inputs.gqa_case(4, 32, 8, 128, [2048, 3000, 4096, 777], seed=1)
    o = _run_gpu(c, want_lse=False)
    got = oracle.bf16_bits_to_f64(bf16_bits(o))
    args = (c.q, c.k, c.v, c.k_scale, c.v_scale, c.cu_seqlens, c.softmax_scale)
    ref = oracle.attn_decode_int8kv(*args, mode="ref")
    deq = oracle.bf16_bits_to_f64(oracle.round_bf16(oracle.attn_decode_int8kv(*args, mode="dequant")))
    n = np.linalg.norm(ref)
    assert np.linalg.norm(got - ref) / n <= np.linalg.norm(deq - ref) / n
    # distance to the untiled definition (global softmax maximum) stays inside the same budget
    glob = oracle.attn_decode_int8kv(*args, mode="global")
    _assert_close(got, glob)


def _subcase(c, seqs):
    """The sub-problem made of the listed sequences only (all heads)."""
    cu = c.cu_seqlens
    tok = np.concatenate([np.arange(cu[b], cu[b + 1]) for b in seqs])
    L = [int(cu[b + 1] - cu[b]) for b in seqs]
    ncu = np.zeros(len(seqs) + 1, np.int32)
    ncu[1:] = np.cumsum(L)
    return inputs.AttnCase(c.q[seqs], c.k[tok], None if c.v is None else c.v[tok], c.k_scale[tok],
                           None if c.v_scale is None else c.v_scale[tok], ncu, c.dv, c.softmax_scale)


def test_gqa_full_size_sampled_sequences():
    """The GQA decode workload at full size (batch 32, 32 query / 8 KV heads, d 128, lengths in [2048, 8192]) in the
    benchmark's launch configuration; the oracle recomputes three sequences."""
    B, Hq, Hkv, D = 32, 32, 8, 128
    c = inputs.gqa_case(B, Hq, Hkv, D, inputs.seqlens_uniform(B, 2048, 8192, seed=0), seed=0)
    o = _run_gpu(c, want_lse=False)
    got = oracle.bf16_bits_to_f64(bf16_bits(o))
    seqs = [0, 17, 31]
    sub = _subcase(c, seqs)
    ref, _ = _oracle_tiled(sub, all_seqlens=np.diff(c.cu_seqlens), seqs=seqs, max_seqlen=c.max_seqlen)
    _assert_close(got[seqs], ref)


def test_mla_full_size_sampled_sequence():
    """The MLA-shaped decode workload at full size (B=64, 64 heads, d=576/512, 16384 tokens); the oracle recomputes one sequence."""
    B, Hq, D, Dv, L = 64, 64, 576, 512, 16384
    c = inputs.mla_case(B, Hq, D, Dv, [L] * B, seed=0)
    o = _run_gpu(c, want_lse=False)
    got = oracle.bf16_bits_to_f64(bf16_bits(o))
    sub = _subcase(c, [37])
    ref, _ = _oracle_tiled(sub, all_seqlens=[L] * B, seqs=[37], max_seqlen=L)
    _assert_close(got[[37]], ref)


def test_kv_dequant_kernel_bit_exact():
    """The cache expansion of the comparison arm: bf16(s * q), FP32 product rounded to nearest even."""
    c = inputs.gqa_case(B=3, Hq=8, Hkv=2, D=128, seqlens=[130, 1, 257], seed=31)
    got = bf16_bits(binding.kv_dequant_bf16(dev(c.k), dev(c.k_scale)))
    prod = (c.k_scale[:, :, None].astype(np.float32) * c.k.astype(np.float32)).astype(np.float64)
    want = oracle.round_bf16(prod)
    assert np.array_equal(got.view(np.uint16), want.view(np.uint16))
    empty = binding.kv_dequant_bf16(dev(c.k[:0]), dev(c.k_scale[:0]))
    assert empty.shape[0] == 0


def test_dequant_bf16_comparison_arm_is_less_accurate():
    """The arm MSD replaces (Sec. 6.4 "Dequant"): our expansion kernel, then a library BF16 attention.  It follows the
    oracle's dequantize-to-BF16 mode, and against the FP64 reference on the dequantized cache it is no better than
    the MSD kernel."""
    c = inputs.gqa_case(B=2, Hq=8, Hkv=2, D=128, seqlens=[700, 333], seed=32)
    kb = binding.kv_dequant_bf16(dev(c.k), dev(c.k_scale))
    vb = binding.kv_dequant_bf16(dev(c.v), dev(c.v_scale))
    q = bf16_dev(c.q)
    outs = []
    for b in range(2):
        t0, t1 = int(c.cu_seqlens[b]), int(c.cu_seqlens[b + 1])
        o = torch.nn.functional.scaled_dot_product_attention(
            q[b][None, :, None, :], kb[t0:t1].permute(1, 0, 2)[None], vb[t0:t1].permute(1, 0, 2)[None],
            scale=c.softmax_scale, enable_gqa=True)
        outs.append(o[0, :, 0, :])
    got = oracle.bf16_bits_to_f64(bf16_bits(torch.stack(outs)))
    deq = oracle.attn_decode_int8kv(c.q, c.k, c.v, c.k_scale, c.v_scale, c.cu_seqlens, c.softmax_scale, dv=c.dv, mode="dequant")
    ref = oracle.attn_decode_int8kv(c.q, c.k, c.v, c.k_scale, c.v_scale, c.cu_seqlens, c.softmax_scale, dv=c.dv, mode="ref")
    n = np.linalg.norm(ref, axis=-1, keepdims=True)
    assert np.all(np.abs(got - deq) <= 1e-2 * n)          # library summation order and P rounding differ from the oracle's
    msd = oracle.bf16_bits_to_f64(bf16_bits(_run_gpu(c)[0]))
    assert np.linalg.norm(msd - ref) <= np.linalg.norm(got - ref) * 1.05


@pytest.mark.parametrize("B,Hq,Hkv,D,seqlens", [
    (2, 8, 2, 128, [700, 333]), (3, 32, 8, 128, [129, 0, 4000]), (1, 16, 1, 128, [1]), (2, 12, 4, 64, [2049, 128]),
])
def test_bf16_kv_comparison_kernel(B, Hq, Hkv, D, seqlens):
    """The whole comparison arm in our own kernels (Sec. 6.4 "Dequant"): cache expansion to BF16, then BF16 decode
    attention with FP32 accumulation.  It follows the oracle's dequantize-to-BF16 mode (same tolerance as the library
    attention above: summation order and the tile-wise running maximum differ from the oracle's single pass), and
    against the FP64 reference on the dequantized cache it is no better than the MSD kernel."""
    c = inputs.gqa_case(B=B, Hq=Hq, Hkv=Hkv, D=D, seqlens=seqlens, seed=40 + Hq)
    if c.dv != 128:                                    # values of width 128 whatever the key width
        rng = np.random.default_rng(3)
        T = c.k.shape[0]
        c = inputs.AttnCase(c.q, c.k, rng.integers(-127, 128, (T, Hkv, 128), dtype=np.int8), c.k_scale,
                            (rng.random((T, Hkv), dtype=np.float32) * 0.02 + 0.01), c.cu_seqlens, 128, c.softmax_scale)
    kb = binding.kv_dequant_bf16(dev(c.k), dev(c.k_scale))
    vb = binding.kv_dequant_bf16(dev(c.v), dev(c.v_scale))
    o, lse = binding.attn_decode_bf16kv(bf16_dev(c.q), kb, vb, dev(c.cu_seqlens), max(c.max_seqlen, 1), c.softmax_scale, want_lse=True)
    torch.cuda.synchronize()
    binding.last_device_status()
    got = oracle.bf16_bits_to_f64(bf16_bits(o))
    args = (c.q, c.k, c.v, c.k_scale, c.v_scale, c.cu_seqlens, c.softmax_scale)
    deq, lse_ref = oracle.attn_decode_int8kv(*args, dv=c.dv, mode="dequant", want_lse=True)
    ref = oracle.attn_decode_int8kv(*args, dv=c.dv, mode="ref")
    n = np.linalg.norm(ref, axis=-1, keepdims=True)
    assert np.all(np.abs(got - deq) <= 1e-2 * n + 1e-30)
    live = np.isfinite(lse_ref)
    assert np.allclose(lse.cpu().numpy()[live], lse_ref[live], rtol=0, atol=2e-3)
    assert np.all(np.isneginf(lse.cpu().numpy()[~live])) and np.all(got[~live] == 0)
    msd = oracle.bf16_bits_to_f64(bf16_bits(_run_gpu(c)[0]))
    assert np.linalg.norm(msd - ref) <= np.linalg.norm(got - ref) * 1.05
    with pytest.raises(binding.MsdError):             # shapes the comparison kernel does not take
        binding.attn_decode_bf16kv(bf16_dev(c.q), kb, vb[:, :, :64].contiguous(), dev(c.cu_seqlens), max(c.max_seqlen, 1), c.softmax_scale)


@pytest.mark.parametrize("page", [16, 64, 128, -64])
def test_paged_cache_gqa(page):
    """The same sequences scattered over a paged cache (random block order, noise in the unused blocks and in the tails
    of the last blocks) must give what the contiguous cache gives: the oracle's tiled mode on the contiguous case."""
    if page < 0:                                      # the same under the balanced split schedule
        binding.debug_set_option("MSD_ATTN_BALANCED", 1)
        page = -page
    seqlens = [1, 130, 700, 0, 257, 2049]
    c = inputs.gqa_case(B=len(seqlens), Hq=16, Hkv=4, D=128, seqlens=seqlens, seed=61)
    k, v, ks, vs, table, sl = inputs.paginate(c, page, seed=page)
    o, lse = binding.attn_decode_int8kv_paged(bf16_dev(c.q), dev(k), dev(v), dev(ks), dev(vs), dev(table), dev(sl), page,
                                              max(c.max_seqlen, 1), c.softmax_scale, want_lse=True)
    torch.cuda.synchronize()
    binding.last_device_status()
    ref, lse_ref = _oracle_tiled(c, paged=True)
    got = oracle.bf16_bits_to_f64(bf16_bits(o))
    live = np.isfinite(lse_ref)
    _assert_close(got[live], ref[live])
    assert np.allclose(lse.cpu().numpy()[live], lse_ref[live], rtol=0, atol=2e-3)
    # and bit for bit what the contiguous entry point returns for the same data
    o2, _ = _run_gpu(c)
    assert torch.equal(o[torch.from_numpy(live).cuda()], o2[torch.from_numpy(live).cuda()])


def test_paged_cache_mla_and_bad_page_size():
    c = inputs.mla_case(B=3, Hq=64, D=576, Dv=512, seqlens=[300, 129, 1000], seed=62)
    k, v, ks, vs, table, sl = inputs.paginate(c, 32, seed=5)
    assert v is None
    o = binding.attn_decode_int8kv_paged(bf16_dev(c.q), dev(k), None, dev(ks), None, dev(table), dev(sl), 32, c.max_seqlen,
                                         c.softmax_scale, dv=c.dv)
    torch.cuda.synchronize()
    binding.last_device_status()
    ref, _ = _oracle_tiled(c, paged=True)
    _assert_close(oracle.bf16_bits_to_f64(bf16_bits(o)), ref)
    with pytest.raises(binding.MsdError):
        binding.attn_decode_int8kv_paged(bf16_dev(c.q), dev(k), None, dev(ks), None, dev(table), dev(sl), 48, c.max_seqlen,
                                         c.softmax_scale, dv=c.dv)


def _truncate(c, drop):
    """The same cache with the last `drop` tokens of every sequence removed (plain indexing)."""
    L = np.diff(c.cu_seqlens)
    keep = np.concatenate([np.arange(c.cu_seqlens[b], c.cu_seqlens[b] + L[b] - drop) for b in range(len(L))]).astype(np.int64)
    cu = np.zeros(len(L) + 1, np.int32)
    cu[1:] = np.cumsum(L - drop)
    return keep, cu


@pytest.mark.parametrize("Sq,Hq,Hkv", [(4, 8, 2), (2, 16, 2), (3, 8, 8), (3, 16, 1), (-3, 8, 8), (-2, 8, 4)])
def test_speculative_decode_rows_are_causal_single_query_problems(Sq, Hq, Hkv):
    """Sq query tokens per sequence: query token s must equal the single-query problem on the cache without the last
    Sq - 1 - s tokens (the oracle, tiled with the kernel's tile and split boundaries)."""
    if Sq < 0:                                        # the same under the balanced split schedule
        binding.debug_set_option("MSD_ATTN_BALANCED", 1)
        Sq = -Sq
    seqlens = [Sq, 131, 700, 2100]
    base = inputs.gqa_case(B=len(seqlens), Hq=Hq * Sq, Hkv=Hkv, D=128, seqlens=seqlens, seed=71)
    B = len(seqlens)
    q = base.q.reshape(B, Sq, Hq, 128)                       # [B,Sq,Hq,D] as the entry point expects
    out, lse = binding.attn_decode_int8kv_spec(bf16_dev(q), dev(base.k), dev(base.v), dev(base.k_scale), dev(base.v_scale),
                                               dev(base.cu_seqlens), base.max_seqlen, base.softmax_scale, want_lse=True)
    torch.cuda.synchronize()
    binding.last_device_status()
    got = oracle.bf16_bits_to_f64(bf16_bits(out))
    starts, tile = _split_starts(base, q_len=Sq)             # [B, Hkv, Sq * Gr, n_splits + 1], rows token-major
    Gr = Hq // Hkv
    for s in range(Sq):
        keep, cu = _truncate(base, Sq - 1 - s)
        ss = np.ascontiguousarray(starts[:, :, s * Gr:(s + 1) * Gr]).reshape(B, Hq, -1)     # (clipped to the shorter cache by the oracle)
        ref, lse_ref = oracle.attn_decode_int8kv(np.ascontiguousarray(q[:, s]), base.k[keep], base.v[keep], base.k_scale[keep],
                                                 base.v_scale[keep], cu, base.softmax_scale, dv=128, tile=tile,
                                                 split_starts=ss, want_lse=True,
                                                 **_softmax_mode(B, Hq * Sq, Hkv, 128, 128, base.max_seqlen))
        _assert_close(got[:, s], ref)
        assert np.allclose(lse.cpu().numpy()[:, s], lse_ref, rtol=0, atol=2e-3)


# ---- Alg. 3 lines 1-4 bit for bit: query components, their scales and both INT32 score planes -------------------------
def _dump_buffers(rows, rows_per_seq, D, T):
    q_dbg = torch.full((2, rows, D), 99, dtype=torch.int8, device="cuda")
    qs_dbg = torch.full((2, rows), -1.0, dtype=torch.float32, device="cuda")
    s_dbg = torch.full((2, rows_per_seq, max(T, 1)), -(2 ** 31), dtype=torch.int32, device="cuda")
    return q_dbg, qs_dbg, s_dbg


def _check_q_dump(q_bits_rows, q_dbg, qs_dbg, live=None):
    """q_bits_rows [R, D]: every query row in the order the entry point takes them; live: rows whose sequence is not
    empty (an empty sequence has no attention to compute and its rows are not decomposed)."""
    o1, o2, oa, ob = oracle.decompose_int8(q_bits_rows)
    live = slice(None) if live is None else live
    assert np.array_equal(q_dbg[0].cpu().numpy()[live], o1[live]) and np.array_equal(q_dbg[1].cpu().numpy()[live], o2[live])
    assert np.array_equal(qs_dbg[0].cpu().numpy()[live], oa[live]) and np.array_equal(qs_dbg[1].cpu().numpy()[live], ob[live])


def _run_with_dump(fn, rows, rows_per_seq, D, T):
    q_dbg, qs_dbg, s_dbg = _dump_buffers(rows, rows_per_seq, D, T)
    binding.debug_set_attn_dump(q_dbg, qs_dbg, s_dbg)
    try:
        fn()
        torch.cuda.synchronize()
        binding.last_device_status()
    finally:
        binding.debug_set_attn_dump()
    return q_dbg, qs_dbg, s_dbg.cpu().numpy()


@pytest.mark.parametrize("kind", ["gqa_narrow", "gqa_8", "gqa_7_d64", "gqa_8_balanced", "gqa_16", "mla"])
def test_query_components_and_scores_bit_exact(kind):
    """North-star requirement: decomposed components, scales and INT32 accumulators bit-exact.  The kernels dump what
    they computed (msd_debug_set_attn_dump); the oracle returns the same planes (Alg. 3 lines 1-4)."""
    if kind == "gqa_narrow":
        c = inputs.gqa_case(3, 8, 2, 128, [700, 64, 1500], seed=41)          # rows decomposed inside the attention CTAs
    elif kind == "gqa_8":
        c = inputs.gqa_case(3, 16, 2, 128, [700, 64, 1500], seed=45)         # 8 rows: a warp decomposes two, 16 lanes each
    elif kind == "gqa_7_d64":
        c = inputs.gqa_case(2, 14, 2, 64, [300, 129], seed=46)               # an odd row count, half a chunk of d
    elif kind == "gqa_8_balanced":
        binding.debug_set_option("MSD_ATTN_BALANCED", 1)                     # rows decomposed again in every segment
        c = inputs.gqa_case(5, 16, 2, 128, [200, 0, 1100, 64, 900], seed=47)
    elif kind == "gqa_16":
        c = inputs.gqa_case(2, 32, 2, 128, [513, 2222], seed=42)            # 16 rows per KV head
    else:
        c = inputs.mla_case(2, 64, 576, 512, [300, 1000], seed=43)          # 64 rows: decomposed by the query-stack kernel
    B, Hq, D = c.q.shape
    T = c.k.shape[0]
    q_dbg, qs_dbg, s_dbg = _run_with_dump(lambda: _run_gpu(c, want_lse=False), B * Hq, Hq, D, T)
    _check_q_dump(c.q.reshape(B * Hq, D), q_dbg, qs_dbg, live=np.repeat(np.diff(c.cu_seqlens) > 0, Hq))
    _, s_ref = oracle.attn_decode_int8kv(c.q, c.k, c.v, c.k_scale, c.v_scale, c.cu_seqlens, c.softmax_scale, dv=c.dv, want_s=True)
    # token t belongs to exactly one sequence, so the plane [row of that sequence, t] is defined for every t
    assert np.array_equal(s_dbg, s_ref)


def test_scores_bit_exact_paged_and_speculative():
    # paged: the dump is indexed by the physical cache row
    seqlens = [130, 700, 0, 257]
    c = inputs.gqa_case(B=len(seqlens), Hq=16, Hkv=4, D=128, seqlens=seqlens, seed=44)
    page = 32
    k, v, ks, vs, table, sl = inputs.paginate(c, page, seed=7)
    B, Hq, D = c.q.shape
    q_dbg, qs_dbg, s_dbg = _run_with_dump(
        lambda: binding.attn_decode_int8kv_paged(bf16_dev(c.q), dev(k), dev(v), dev(ks), dev(vs), dev(table), dev(sl), page,
                                                 max(c.max_seqlen, 1), c.softmax_scale), B * Hq, Hq, D, k.shape[0])
    _check_q_dump(c.q.reshape(B * Hq, D), q_dbg, qs_dbg, live=np.repeat(np.asarray(seqlens) > 0, Hq))
    _, s_ref = oracle.attn_decode_int8kv(c.q, c.k, c.v, c.k_scale, c.v_scale, c.cu_seqlens, c.softmax_scale, dv=c.dv, want_s=True)
    for b in range(B):
        for u in range(seqlens[b]):
            row = table[b, u // page] * page + u % page
            assert np.array_equal(s_dbg[:, :, row], s_ref[:, :, c.cu_seqlens[b] + u])
    # speculative decode: rows are (query token, head); every row's sums against EVERY token of its sequence are dumped
    Sq, Hq, Hkv = 3, 8, 2
    seqlens = [Sq, 131, 700]
    base = inputs.gqa_case(B=len(seqlens), Hq=Hq * Sq, Hkv=Hkv, D=128, seqlens=seqlens, seed=45)
    B = len(seqlens)
    q = base.q.reshape(B, Sq, Hq, 128)
    T = base.k.shape[0]
    q_dbg, qs_dbg, s_dbg = _run_with_dump(
        lambda: binding.attn_decode_int8kv_spec(bf16_dev(q), dev(base.k), dev(base.v), dev(base.k_scale), dev(base.v_scale),
                                                dev(base.cu_seqlens), base.max_seqlen, base.softmax_scale),
        B * Sq * Hq, Sq * Hq, 128, T)
    _check_q_dump(q.reshape(B * Sq * Hq, 128), q_dbg, qs_dbg)
    for s in range(Sq):
        _, s_ref = oracle.attn_decode_int8kv(np.ascontiguousarray(q[:, s]), base.k, base.v, base.k_scale, base.v_scale,
                                             base.cu_seqlens, base.softmax_scale, dv=128, want_s=True)
        assert np.array_equal(s_dbg[:, s * Hq:(s + 1) * Hq], s_ref)


def test_latent_head_of_384_with_aliased_values():
    """D = Dv = 384 with V aliased to the K rows: three 128-byte chunks are loaded per tile while PV is computed as four
    128-wide tiles, so the KV stage must be sized for four."""
    c = inputs.mla_case(2, 8, 384, 384, [300, 129], seed=46)
    _check(c)
    c = inputs.mla_case(1, 32, 320, 320, [700], seed=47)
    _check(c)
