"""The KV-cache structure (appendix "Quantization Dimension", Fig. 9b) on the GPU against its oracle: stored keys and
value chunks bit for bit, the high-precision remainder byte for byte, scores and P V within the product tolerance,
under token-by-token and bulk appends."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_01144_b200 as bd
from oracle.kvcache import KVCache as OracleCache
from paper_2501_01144_b200 import inputs
from util import ORACLE_DTYPE, gemm_tolerance_ok, to_device

pytestmark = pytest.mark.gpu


def _rows(n, d, kind, seed):
    rng = np.random.default_rng(seed)
    k = rng.standard_normal((n, d)).astype(np.float32)
    k[:, rng.integers(0, d)] *= 12.0
    v = (rng.standard_normal((n, d)) * np.exp2(rng.integers(-3, 4, (1, d)))).astype(np.float32)
    if kind == torch.float32:
        return k, v
    if kind == torch.bfloat16:
        return inputs.to_bf16_bits(k), inputs.to_bf16_bits(v)
    return inputs.to_f16_bits(k), inputs.to_f16_bits(v)


def _stored_values(cache, n_q):
    """Canonical view of the first n_q tokens of the library's value operand [head_dim, n_q]."""
    codes, ids, scales = (t.cpu().numpy() for t in bd.export_canonical(cache.v))
    return codes[:, :n_q // 2], ids[:, :n_q // 32], scales[:, :n_q // 32]


def _check_state(cache, ref, kind):
    n, n_q = ref.length, ref.length // 32 * 32
    assert cache.length == n
    kc, ki, ks = (t.cpu().numpy()[:n] for t in bd.export_canonical(cache.k))
    rc, ri, rs = ref.keys()
    assert np.array_equal(ks, rs) and np.array_equal(ki, ri) and np.array_equal(kc, rc), "stored keys"
    if n_q:
        got, want = _stored_values(cache, n_q), ref.values_quantised()
        assert all(np.array_equal(g, w) for g, w in zip(got, want)), "stored value chunks"
    r = n - n_q
    if r:
        recent = cache.v_recent[:r].float().cpu().numpy().astype(np.float64)
        assert np.array_equal(recent, ref.values_recent()), "high-precision remainder"


@pytest.mark.parametrize("kind", [torch.bfloat16, torch.float32, torch.float16])
@pytest.mark.parametrize("d", [64, 128])
def test_appends_in_uneven_pieces_match_the_oracle(kind, d):
    total, cap = 333, 512
    k, v = _rows(total, d, kind, seed=d + 1)
    cache, ref = bd.KVCache(cap, d, dtype=kind), OracleCache(d, dtype=ORACLE_DTYPE[kind])
    pos = 0
    for t in (1, 1, 29, 1, 1, 40, 64, 3, 100, 31, 32, 30):            # crossing chunk borders in every way
        cache.append(to_device(k[pos:pos + t], kind), to_device(v[pos:pos + t], kind))
        ref.append(k[pos:pos + t], v[pos:pos + t])
        pos += t
        _check_state(cache, ref, kind)
    assert pos == total
    bd.poll_status()


@pytest.mark.parametrize("n,q_rows", [(19, 4), (32, 1), (77, 4), (1000, 8), (4096, 4), (4127, 130)])
def test_scores_and_pv_match_the_oracle(n, q_rows):
    d, cap, kind = 128, 4160, torch.bfloat16
    k, v = _rows(n, d, kind, seed=n)
    cache, ref = bd.KVCache(cap, d, dtype=kind), OracleCache(d)
    cache.append(to_device(k, kind), to_device(v, kind))
    ref.append(k, v)
    _check_state(cache, ref, kind)
    rng = np.random.default_rng(n + q_rows)
    qb = inputs.to_bf16_bits(rng.standard_normal((q_rows, d)).astype(np.float32))
    Qq = bd.quantize_act(to_device(qb, torch.bfloat16))
    S = cache.scores(Qq).cpu().numpy()
    Sref, T = ref.scores(oracle.quantize(qb, dtype=oracle.BF16))
    ok, ratio = gemm_tolerance_ok(S, Sref, T)
    assert ok, f"scores: max err / bound = {ratio}"
    # probabilities: softmax of the library's own scores in fp64, handed in as fp32 (softmax stays in high precision)
    z = S.astype(np.float64) / np.sqrt(d)
    P = np.exp(z - z.max(-1, keepdims=True))
    P = (P / P.sum(-1, keepdims=True)).astype(np.float32)
    Pd = torch.zeros(q_rows, (n + 3) // 4 * 4, device="cuda")[:, :n]          # a row pitch of whole 16 bytes
    Pd.copy_(torch.from_numpy(P))
    O = cache.pv(Pd).cpu().numpy()
    Oref, To = ref.pv(P)
    ok, ratio = gemm_tolerance_ok(O, Oref, To)
    assert ok, f"P V: max err / bound = {ratio}"
    O16 = cache.pv(Pd, dtype=torch.bfloat16)
    assert torch.equal(O16.cpu(), torch.from_numpy(O).to(torch.bfloat16))
    bd.poll_status()


def test_decoding_token_by_token_never_changes_a_stored_chunk():
    d, kind = 64, torch.bfloat16
    k, v = _rows(100, d, kind, seed=9)
    cache = bd.KVCache(128, d, dtype=kind)
    cache.append(to_device(k[:64], kind), to_device(v[:64], kind))
    before = [np.array(b) for b in _stored_values(cache, 64)]
    for t in range(64, 100):
        cache.append(to_device(k[t:t + 1], kind), to_device(v[t:t + 1], kind))
    after = _stored_values(cache, 64)
    assert all(np.array_equal(a, b) for a, b in zip(after, before))
    with pytest.raises(bd.BdError):
        cache.append(to_device(k[:64], kind), to_device(v[:64], kind))       # beyond the capacity
    bd.poll_status()


@pytest.mark.parametrize("n,q_rows,heads,d", [(19, 4, 3, 128), (77, 4, 8, 128), (1000, 8, 2, 64), (4127, 4, 8, 128), (300, 12, 3, 128)])
@pytest.mark.parametrize("impl", [bd.GEMM_AUTO, bd.GEMM_SIMT])
def test_batched_heads_match_the_oracle_head_by_head(n, q_rows, heads, d, impl):
    # the KV heads of a layer in one call (one launch sequence for all heads with at most 16 query rows, head by head
    # otherwise): every head against its own oracle cache, guard bands around results and workspace strides
    cap, kind = 4160, torch.bfloat16
    caches, refs, Qs, Qrefs = [], [], [], []
    rng = np.random.default_rng(n + q_rows + heads)
    for h in range(heads):
        k, v = _rows(n, d, kind, seed=n + 7 * h)
        c, r = bd.KVCache(cap, d, dtype=kind), OracleCache(d)
        c.append(to_device(k, kind), to_device(v, kind))
        r.append(k, v)
        caches.append(c)
        refs.append(r)
        qb = inputs.to_bf16_bits(rng.standard_normal((q_rows, d)).astype(np.float32))
        Qs.append(bd.quantize_act(to_device(qb, torch.bfloat16)))
        Qrefs.append(oracle.quantize(qb, dtype=oracle.BF16))
    bd.set_gemm_impl(impl)
    try:
        pitch = (n + 3) // 4 * 4
        S_all = torch.full((heads, q_rows, pitch + 4), -7.0, device="cuda")
        S = S_all[:, :, :n]
        before = bd.launch_count()
        bd.kvcache_scores_batched(caches, Qs, out=S)
        if impl == bd.GEMM_AUTO and q_rows <= 16:
            assert bd.launch_count() - before == 1, "one launch: the product kernel reads the queries' codes itself"
        assert (S_all[:, :, n:] == -7.0).all(), "write past the scores' rows"
        Sh = S.cpu().numpy()
        P = np.zeros((heads, q_rows, n), np.float32)
        for h in range(heads):
            Sref, T = refs[h].scores(Qrefs[h])
            ok, ratio = gemm_tolerance_ok(Sh[h], Sref, T)
            assert ok, f"head {h} scores: max err / bound = {ratio}"
            z = Sh[h].astype(np.float64) / np.sqrt(d)
            e = np.exp(z - z.max(-1, keepdims=True))
            P[h] = (e / e.sum(-1, keepdims=True)).astype(np.float32)
        Pd = torch.zeros(heads, q_rows, pitch, device="cuda")[:, :, :n]
        Pd.copy_(torch.from_numpy(P))
        O_all = torch.full((heads, q_rows, d + 8), -7.0, device="cuda")
        before = bd.launch_count()
        bd.kvcache_pv_batched(caches, Pd, out=O_all[:, :, :d])
        if impl == bd.GEMM_AUTO and q_rows <= 16:
            assert bd.launch_count() - before == (2 if n >= 32 else 1), "records, then the product with the recent tokens in its epilogue"
        assert (O_all[:, :, d:] == -7.0).all(), "write past the result's rows"
        Oh = O_all[:, :, :d].cpu().numpy()
        for h in range(heads):
            Oref, To = refs[h].pv(P[h])
            ok, ratio = gemm_tolerance_ok(Oh[h], Oref, To)
            assert ok, f"head {h} P V: max err / bound = {ratio}"
            # and the single-head call agrees (the shares of K may be cut differently, so not bit for bit)
            ok, ratio = gemm_tolerance_ok(caches[h].pv(Pd[h]).cpu().numpy(), Oref, To)
            assert ok, f"head {h} P V, single call: max err / bound = {ratio}"
        O16 = bd.kvcache_pv_batched(caches, Pd, dtype=torch.bfloat16)
        assert torch.equal(O16.cpu(), torch.from_numpy(Oh).to(torch.bfloat16))
    finally:
        bd.set_gemm_impl(bd.GEMM_AUTO)
    bd.poll_status()


@pytest.mark.parametrize("kind", [torch.bfloat16, torch.float32])
def test_batched_appends_leave_every_head_in_the_oracle_state(kind):
    # the heads of a layer take their new tokens in one call (pieces that cross chunk borders in every way); each
    # head's stored keys, value chunks and high-precision rows against its own oracle cache after every piece
    heads, d, total, cap = 5, 128, 203, 256
    rows = [_rows(total, d, kind, seed=31 + h) for h in range(heads)]
    caches = [bd.KVCache(cap, d, dtype=kind) for _ in range(heads)]
    refs = [OracleCache(d, dtype=ORACLE_DTYPE[kind]) for _ in range(heads)]
    pos = 0
    for t in (1, 30, 1, 1, 64, 3, 40, 31, 32):
        k_new = torch.stack([to_device(rows[h][0][pos:pos + t], kind) for h in range(heads)])
        v_new = torch.stack([to_device(rows[h][1][pos:pos + t], kind) for h in range(heads)])
        before = bd.launch_count()
        bd.kvcache_append_batched(caches, k_new, v_new)
        assert bd.launch_count() - before <= 5, "the heads share their launches"
        for h in range(heads):
            refs[h].append(rows[h][0][pos:pos + t], rows[h][1][pos:pos + t])
            _check_state(caches[h], refs[h], kind)
        pos += t
    assert pos == total
    bd.poll_status()


@pytest.mark.parametrize("n,q_rows,heads,d", [(19, 4, 2, 128), (77, 1, 4, 64), (1000, 8, 3, 128), (4127, 4, 8, 128), (640, 12, 2, 128)])
def test_decode_step_attention_link_by_link(n, q_rows, heads, d):
    # scores -> fp32 softmax -> P V in one call.  The probabilities come back through the optional output: they are
    # held against the oracle's fp64 softmax of its own scores, and the result against the oracle's P V of the
    # LIBRARY's probabilities (a probability that differs in its last bit may round to another code, which is a
    # different, equally valid, input to the second product); the call without the output buffer gives the same result
    cap, kind, scale = 4160, torch.bfloat16, 1.0 / np.sqrt(d)
    caches, refs, Qs, Qrefs = [], [], [], []
    rng = np.random.default_rng(n + q_rows)
    for h in range(heads):
        k, v = _rows(n, d, kind, seed=n + 11 * h)
        c, r = bd.KVCache(cap, d, dtype=kind), OracleCache(d)
        c.append(to_device(k, kind), to_device(v, kind))
        r.append(k, v)
        caches.append(c)
        refs.append(r)
        qb = inputs.to_bf16_bits(rng.standard_normal((q_rows, d)).astype(np.float32))
        Qs.append(bd.quantize_act(to_device(qb, torch.bfloat16)))
        Qrefs.append(oracle.quantize(qb, dtype=oracle.BF16))
    pitch = (n + 3) // 4 * 4
    probs_all = torch.full((heads, q_rows, pitch + 4), -7.0, device="cuda")
    probs = probs_all[:, :, :pitch]
    before = bd.launch_count()
    O = bd.kvcache_attention(caches, Qs, scale, probs=probs).cpu().numpy()
    assert bd.launch_count() - before == 3, "scores, softmax with the records, product"
    assert (probs_all[:, :, pitch:] == -7.0).all()
    P = probs[:, :, :n].cpu().numpy()
    for h in range(heads):
        _, _, Pref = refs[h].attention(Qrefs[h], scale)
        assert np.abs(P[h].astype(np.float64) - Pref.astype(np.float64)).max() <= 2e-6, f"head {h}: probabilities"
        assert np.abs(P[h].astype(np.float64).sum(-1) - 1.0).max() <= 1e-5
        Oref, To = refs[h].pv(P[h])
        ok, ratio = gemm_tolerance_ok(O[h], Oref, To)
        assert ok, f"head {h}: P V of the library's probabilities: max err / bound = {ratio}"
    O2 = bd.kvcache_attention(caches, Qs, scale).cpu().numpy()
    for h in range(heads):
        Oref, To = refs[h].pv(P[h])
        ok, ratio = gemm_tolerance_ok(O2[h], Oref, To)
        assert ok, f"head {h}: without the probabilities' buffer: max err / bound = {ratio}"
    O16 = bd.kvcache_attention(caches, Qs, scale, dtype=torch.bfloat16)
    assert torch.equal(O16.cpu(), torch.from_numpy(O2).to(torch.bfloat16))
    bd.poll_status()


def test_decode_loop_appends_and_attends_back_to_back():
    # token by token: the new token of every head is appended and the step's attention follows at once on the same
    # stream, with nothing in between (the scores kernel's copies of the key cache must wait for the append kernels);
    # every step's result against the oracle caches, which take the same tokens
    heads, d, kind, start, steps = 3, 128, torch.bfloat16, 50, 40
    scale = 1.0 / np.sqrt(d)
    rows = [_rows(start + steps, d, kind, seed=71 + h) for h in range(heads)]
    caches = [bd.KVCache(128, d, dtype=kind) for _ in range(heads)]
    refs = [OracleCache(d) for _ in range(heads)]
    for h in range(heads):
        caches[h].append(to_device(rows[h][0][:start], kind), to_device(rows[h][1][:start], kind))
        refs[h].append(rows[h][0][:start], rows[h][1][:start])
    rng = np.random.default_rng(3)
    qb = [inputs.to_bf16_bits(rng.standard_normal((steps, 2, d)).astype(np.float32)) for _ in range(heads)]
    k_all = torch.stack([to_device(rows[h][0][start:], kind) for h in range(heads)])      # [heads, steps, d]
    v_all = torch.stack([to_device(rows[h][1][start:], kind) for h in range(heads)])
    Qs_all = [[bd.quantize_act(to_device(qb[h][t], torch.bfloat16)) for h in range(heads)] for t in range(steps)]
    outs, probs = [], []
    torch.cuda.synchronize()
    for t in range(steps):                                        # no synchronisation inside the loop
        bd.kvcache_append_batched(caches, k_all[:, t:t + 1], v_all[:, t:t + 1])
        n = start + t + 1
        p = torch.zeros(heads, 2, (n + 3) // 4 * 4, device="cuda")
        outs.append(bd.kvcache_attention(caches, Qs_all[t], scale, probs=p))
        probs.append(p)
    torch.cuda.synchronize()
    for t in range(steps):
        n = start + t + 1
        for h in range(heads):
            refs[h].append(rows[h][0][n - 1:n], rows[h][1][n - 1:n])
            P = probs[t][h, :, :n].cpu().numpy()
            _, _, Pref = refs[h].attention(oracle.quantize(qb[h][t], dtype=oracle.BF16), scale)
            assert np.abs(P.astype(np.float64) - Pref.astype(np.float64)).max() <= 2e-6, f"step {t} head {h}: probabilities"
            Oref, To = refs[h].pv(P)
            ok, ratio = gemm_tolerance_ok(outs[t][h].cpu().numpy(), Oref, To)
            assert ok, f"step {t} head {h}: max err / bound = {ratio}"
    for h in range(heads):
        _check_state(caches[h], refs[h], kind)
    bd.poll_status()
