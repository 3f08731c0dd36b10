"""Host ends of the path (no GPU): keep rate on the target tokenisation (Section 3.1) and ConcatWithDelim
(Algorithm 1, Section 3.2, Appendix A.3).  The oracle's versions are pinned by examples worked by hand; the
library's host routines are then compared with the oracle through the C ABI."""
import random

import numpy as np
import pytest

import oracle


@pytest.fixture(scope="module")
def spf():
    from paper_2603_02631_b200.build import build_library
    build_library()
    import paper_2603_02631_b200 as mod
    return mod


# ------------------------------------------------------------------------------------------- oracle pins
def test_oracle_keep_rate_matches_the_papers_budgets():
    # Section 3.1 / Figure 1: a 128k-token prompt compressed to 16k tokens is a keep rate of 12.5 %
    assert oracle.keep_rate(131072, 16384) == 0.125
    assert oracle.keep_rate(128 * 1024, 32 * 1024) == 0.25
    assert oracle.keep_rate(1000, 5000) == 1.0            # never more than the whole prompt
    assert oracle.keep_rate(0, 10) == 0.0 and oracle.keep_rate(10, 0) == 0.0


def test_oracle_snap_budget_is_whole_blocks():
    # compressed lengths are multiples of the 4k-token KV block: 8k, 16k, 24k, 32k
    assert [oracle.snap_budget(x, 4096) for x in (8192, 16384, 24576, 32768)] == [8192, 16384, 24576, 32768]
    assert oracle.snap_budget(17000, 4096) == 16384
    assert oracle.snap_budget(4095, 4096) == 4096         # at least one block
    assert oracle.snap_budget(0, 4096) == 0


def test_oracle_concat_hand_example():
    text = "The quick brown fox jumps over the lazy dog"
    #       0123456789...            "quick" = [4,9), "fox jumps" = [16,25), "dog" = [40,43)
    assert oracle.concat_with_delim(text, [(4, 9), (16, 25), (40, 43)], "[...]") == "quick[...]fox jumps[...]dog"
    assert oracle.concat_with_delim(text, [(0, len(text))], "[...]") == text          # one span: no delimiter
    assert oracle.concat_with_delim(text, [], "[...]") == ""
    assert oracle.concat_with_delim(text, [(4, 9), (9, 9), (10, 15)], "|") == "quick||brown"   # an empty span still separates
    # characters are code points, not bytes
    assert oracle.concat_with_delim("aé你😀z", [(1, 3), (3, 5)], " // omitted ") == "é你 // omitted 😀z"


# ------------------------------------------------------------------------------------------- library vs oracle
def test_library_keep_rate_and_budget(spf):
    rng = random.Random(5)
    for _ in range(500):
        t, b = rng.randint(-2, 300000), rng.randint(-2, 40000)
        assert spf.spf_keep_rate(t, b) == oracle.keep_rate(t, b)
        blk = rng.choice([1, 16, 4096, 5000])
        assert spf.spf_snap_budget(b, blk) == oracle.snap_budget(b, blk)
    assert spf.spf_snap_budget(17000) == 16384


def _random_text(rng, n):
    alphabet = "abc xyz\n\t.,;(){}" + "éüñßøÆ" + "你好世界漢字" + "😀🚀𝔘" + "́‍"
    return "".join(rng.choice(alphabet) for _ in range(n))


def test_library_concat_matches_oracle_on_random_unicode(spf):
    rng = random.Random(11)
    for trial in range(200):
        n = rng.randint(0, 300)
        text = _random_text(rng, n)
        cuts = sorted(rng.randint(0, n) for _ in range(2 * rng.randint(0, 8)))
        spans = [(cuts[i], cuts[i + 1]) for i in range(0, len(cuts), 2)]
        delim = rng.choice(["[...]", "// omitted", "", " … "])
        assert spf.spf_concat_with_delim(text, spans, delim) == oracle.concat_with_delim(text, spans, delim)


def test_library_concat_on_spans_from_the_selection(spf):
    """Spans as spf_compact_spans emits them: token offsets of a synthetic prompt, merged chunks."""
    rng = np.random.default_rng(3)
    n_tok, chunk = 1000, 32
    lens = rng.integers(1, 9, n_tok)
    start = np.concatenate([[0], np.cumsum(lens)[:-1]]); end = start + lens
    text = _random_text(random.Random(4), int(end[-1]))
    kept = np.sort(rng.choice((n_tok + chunk - 1) // chunk, 9, replace=False))
    _, _, _, char_spans = oracle.compact(kept, chunk, n_tok, np.arange(n_tok), start, end)
    got = spf.spf_concat_with_delim(text, char_spans, "[...]")
    assert got == oracle.concat_with_delim(text, char_spans, "[...]")
    assert got.count("[...]") >= len(char_spans) - 1


def test_library_concat_rejects_bad_spans(spf):
    for spans in ([(5, 3)], [(0, 4), (3, 6)], [(0, 100)], [(-1, 2)]):
        with pytest.raises(spf.SpfError):
            spf.spf_concat_with_delim("hello world", spans, "|")
    # capacity query and short buffer: nothing written, size returned
    import ctypes
    raw = "héllo".encode()
    spans = np.array([[0, 5]], dtype=np.int32)
    buf = ctypes.create_string_buffer(b"\xAA" * 8, 8)
    need = spf.lib.spf_concat_with_delim(raw, len(raw), spans.ctypes.data, 1, b"", 0, buf, 3)
    assert need == 6 and buf.raw == b"\xAA" * 8
