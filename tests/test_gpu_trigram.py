"""GPU parity of the tri-gram store against the CPU checker: counts and top-k lists bit-exact."""
import numpy as np
import pytest
import torch

from oracle.trigram import TrigramStore
from paper_2407_12021_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def _topk_gpu(B, t, ctx, k):
    q = len(ctx)
    c = torch.tensor(ctx, dtype=torch.int32, device="cuda").reshape(q, 2)
    tok = torch.empty((q, k), dtype=torch.int32, device="cuda")
    cnt = torch.empty((q, k), dtype=torch.int32, device="cuda")
    tot = torch.empty((q,), dtype=torch.int32, device="cuda")
    B.aded_trigram_topk(t, c, k, tok, cnt, tot)
    torch.cuda.synchronize()
    return tok.tolist(), cnt.tolist(), tot.tolist()


def _check_against(B, t, st: TrigramStore, contexts, ks=(1, 4, 32)):
    for k in ks:
        tok, cnt, tot = _topk_gpu(B, t, contexts, k)
        for i, (a, b) in enumerate(contexts):
            wt, wc = st.topk(a, b, k)
            assert tok[i] == wt and cnt[i] == wc, (a, b, k, tok[i], wt, cnt[i], wc)
            assert tot[i] == st.total(a, b)


def test_c1_table_from_10k_zipf_corpus(cuda_device):
    """Workload 1's table: 10k-token Zipf(1.1) corpus over a 4096-token vocabulary, k = 4."""
    from paper_2407_12021_b200 import binding as B
    toks = gen.zipf_tokens(10000, 4096, 31, 1)
    st = TrigramStore()
    st.update(toks.tolist())
    t = B.aded_trigram_create(4096, log2_buckets=14, overflow_buckets=4096)
    B.aded_trigram_update(t, toks.cuda())
    torch.cuda.synchronize()
    assert B.aded_trigram_poll_status(t) == 0
    entries, buckets = B.aded_trigram_stats(t)
    assert entries == len(st.entries())
    assert buckets >= len(st.table)
    # every stored tri-gram, bit-exact
    for (a, b, c), n in list(st.entries().items())[::7]:
        assert B.aded_trigram_get(t, a, b, c) == n
    assert B.aded_trigram_get(t, 4095, 4095, 4095) == 0
    ctxs = list(st.table.keys())
    ctxs.sort(key=lambda ab: -len(st.table[ab]))
    contexts = ctxs[:300] + ctxs[-200:] + [(4095, 4094), (7, 4000)]
    _check_against(B, t, st, contexts)


def test_incremental_updates_match_stepwise(cuda_device):
    """The per-step pattern: every step passes [two previous tokens] ++ [new tokens]."""
    from paper_2407_12021_b200 import binding as B
    stream = gen.zipf_tokens(3000, 50, 32, 1).tolist()     # tiny vocabulary: long chains, many duplicates
    st = TrigramStore()
    t = B.aded_trigram_create(50, log2_buckets=12, overflow_buckets=2048)
    pos = 2
    lens = gen.randint(2000, 9, 32, 2)
    i = 0
    while pos < len(stream):
        n = 1 + lens[i]; i += 1
        span = stream[pos - 2:pos + n]
        st.update(span)
        B.aded_trigram_update_host(t, torch.tensor(span, dtype=torch.int32))
        pos += n
    assert B.aded_trigram_poll_status(t) == 0
    whole = TrigramStore()
    whole.update(stream)
    assert whole.entries() == st.entries()
    assert B.aded_trigram_stats(t)[0] == len(st.entries())
    _check_against(B, t, st, list(st.table.keys())[:400])


def test_duplicates_in_one_call_saturation_and_short_spans(cuda_device):
    from paper_2407_12021_b200 import binding as B
    t = B.aded_trigram_create(10, log2_buckets=4, overflow_buckets=64, cap=5)
    st = TrigramStore(cap=5)
    span = [3] * 40 + [1, 2] * 30
    st.update(span)
    B.aded_trigram_update(t, torch.tensor(span, dtype=torch.int32, device="cuda"))
    for n in (0, 1, 2):
        B.aded_trigram_update(t, torch.tensor(span[:n], dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert B.aded_trigram_get(t, 3, 3, 3) == 5 == st.count(3, 3, 3)
    assert B.aded_trigram_get(t, 1, 2, 1) == 5
    assert B.aded_trigram_get(t, 3, 3, 1) == 1
    _check_against(B, t, st, [(3, 3), (1, 2), (2, 1), (3, 1), (9, 9)], ks=(1, 3))


def test_min_count_filter_and_errors(cuda_device):
    from paper_2407_12021_b200 import binding as B
    t = B.aded_trigram_create(100, log2_buckets=6, overflow_buckets=8, min_count=2)
    st = TrigramStore()
    span = [1, 1, 9, 1, 1, 3, 1, 1, 7, 1, 1, 7]
    st.update(span)
    B.aded_trigram_update(t, torch.tensor(span, dtype=torch.int32, device="cuda"))
    tok, cnt, tot = _topk_gpu(B, t, [(1, 1)], 4)
    assert (tok[0], cnt[0]) == st.topk(1, 1, 4, min_count=2) and tot[0] == st.total(1, 1)
    # an out-of-vocabulary token is reported, not counted
    B.aded_trigram_update(t, torch.tensor([1, 2, 100], dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert B.aded_trigram_poll_status(t) == 1
    assert B.aded_trigram_poll_status(t) == 0
    # table full: 64 home buckets cannot hold 90 distinct contexts
    full = B.aded_trigram_create(100, log2_buckets=4, overflow_buckets=0)
    B.aded_trigram_update(full, torch.arange(0, 92, dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert B.aded_trigram_poll_status(full) == 4


def test_large_table_bulk_update_and_queries(cuda_device):
    """10^6 Zipf tokens over a 32000-token vocabulary; sampled contexts against the checker."""
    from paper_2407_12021_b200 import binding as B
    toks = gen.zipf_tokens(1_000_000, 32000, 33, 1)
    st = TrigramStore()
    st.update(toks.tolist())
    t = B.aded_trigram_create(32000, log2_buckets=21, overflow_buckets=1 << 18)
    B.aded_trigram_update(t, toks.cuda())
    torch.cuda.synchronize()
    assert B.aded_trigram_poll_status(t) == 0
    assert B.aded_trigram_stats(t)[0] == len(st.entries())
    ctxs = list(st.table.keys())
    ctxs.sort(key=lambda ab: -len(st.table[ab]))
    sample = ctxs[:64] + ctxs[1000::997][:400]
    _check_against(B, t, st, sample, ks=(4,))


def _entries_gpu(B, t, min_count=0):
    keys, counts = B.aded_trigram_export(t, min_count)
    torch.cuda.synchronize()
    k, c = keys.cpu().tolist(), counts.cpu().tolist()
    out = {tuple(kk): cc for kk, cc in zip(k, c)}
    assert len(out) == len(k), "an entry was exported twice"
    return out


def test_export_prune_save_load(cuda_device, tmp_path):
    """Table persistence and the elimination threshold: exported entries, the pruned table and a table
    read back from a file equal the checker's, bit for bit; the pruned table keeps working."""
    from paper_2407_12021_b200 import binding as B
    vocab = 60
    toks = gen.zipf_tokens(6000, vocab, 41, 1)
    st = TrigramStore(cap=50)
    st.update(toks.tolist())
    t = B.aded_trigram_create(vocab, log2_buckets=12, overflow_buckets=4096, cap=50)
    B.aded_trigram_update(t, toks.cuda())
    assert _entries_gpu(B, t) == st.entries()
    assert _entries_gpu(B, t, 12) == {k: n for k, n in st.entries().items() if n >= 12}
    path = str(tmp_path / "table.bin")
    B.aded_trigram_save(t, path)
    # a copy read from the file
    t2 = B.aded_trigram_create(vocab, log2_buckets=13, overflow_buckets=8192, cap=50)   # another geometry than the source
    B.aded_trigram_load(t2, path)
    assert _entries_gpu(B, t2) == st.entries()
    # loading again adds the counts (saturating)
    B.aded_trigram_load(t2, path)
    twice = TrigramStore(cap=50)
    twice.merge(st.entries())
    twice.merge(st.entries())
    assert _entries_gpu(B, t2) == twice.entries()
    # a file for another vocabulary is refused
    from paper_2407_12021_b200.binding import AdedError
    t3 = B.aded_trigram_create(vocab + 1, log2_buckets=10, overflow_buckets=64)
    with pytest.raises(AdedError):
        B.aded_trigram_load(t3, path)
    with pytest.raises(AdedError):
        B.aded_trigram_load(t2, str(tmp_path / "missing.bin"))
    # elimination threshold 12 (the paper's setting): the table is rebuilt from what stays
    _, buckets_before = B.aded_trigram_stats(t)
    B.aded_trigram_prune(t, 12)
    st.prune(12)
    assert _entries_gpu(B, t) == st.entries()
    entries_after, buckets_after = B.aded_trigram_stats(t)
    assert entries_after == len(st.entries()) and buckets_after < buckets_before
    ctxs = list(st.table.keys())[:200] + [(vocab - 1, vocab - 1)]
    _check_against(B, t, st, ctxs, ks=(1, 4))
    # and keeps counting: no duplicate entries appear where pruned ones used to be
    more = gen.zipf_tokens(3000, vocab, 42, 1)
    B.aded_trigram_update(t, more.cuda())
    st.update(more.tolist())
    assert _entries_gpu(B, t) == st.entries()
    B.aded_trigram_clear(t)
    assert _entries_gpu(B, t) == {} and B.aded_trigram_stats(t) == (0, 0)
    assert B.aded_trigram_poll_status(t) == 0 and B.aded_trigram_poll_status(t2) == 0


def test_import_of_duplicate_entries_with_large_counts_saturates(cuda_device):
    """Imported counts may be large and one tri-gram may appear several times in an import: the stored count
    is min(sum, cap) as in the checker's merge, never a wrapped 32-bit sum.  The default cap is 2^31 - 1;
    a cap above it is refused."""
    from paper_2407_12021_b200 import binding as B
    big = 2 ** 31 - 2
    keys, counts, entries = [], [], []
    for i in range(64):                       # 64 tri-grams, each four times in one import, counts near 2^31
        for rep in range(4):
            keys.append([i % 7, i % 5, i])
            counts.append(big - rep)
            entries.append(((i % 7, i % 5, i), big - rep))
    for cap in (0, 1000, 2 ** 31 - 1):
        t = B.aded_trigram_create(100, log2_buckets=8, overflow_buckets=64, cap=cap)
        st = TrigramStore(cap=cap if cap else 2 ** 31 - 1)
        st.update([1, 2, 3, 1, 2, 3])          # an entry that is there before the import
        B.aded_trigram_update(t, torch.tensor([1, 2, 3, 1, 2, 3], dtype=torch.int32, device=cuda_device))
        kt = torch.tensor(keys + [[1, 2, 3]], dtype=torch.int32, device=cuda_device)
        ct = torch.tensor([c - 2 ** 32 if c >= 2 ** 31 else c for c in counts + [big]], dtype=torch.int32, device=cuda_device)
        B.aded_trigram_import(t, kt, ct)
        for key, n in entries + [((1, 2, 3), big)]:
            st.merge({key: n})
        torch.cuda.synchronize()
        assert B.aded_trigram_poll_status(t) == 0
        for i in range(64):
            assert B.aded_trigram_get(t, i % 7, i % 5, i) == st.count(i % 7, i % 5, i) == st.cap
        assert B.aded_trigram_get(t, 1, 2, 3) == st.count(1, 2, 3) == st.cap
        assert B.aded_trigram_get(t, 2, 3, 1) == st.count(2, 3, 1) == 1
    with pytest.raises(B.AdedError) as err:
        B.aded_trigram_create(100, log2_buckets=8, overflow_buckets=64, cap=2 ** 31)
    assert err.value.status == 1
