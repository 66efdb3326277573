"""Fragment tokenisation (Sec. 3.2): pins for the oracle, and the library's cut points
against it (integer work: identical)."""
import numpy as np
import pytest

from oracle import efim_fragment_oracle as fo
from paper_2505_21889_b200 import fragment as fr

VOCAB = ["def ", "return ", "self", "model", "models", "comp", "lete", "complete", "code ", "(", ")", ":", "\n", "    "]


def toy_tokenize(text):
    """Greedy longest match over a tiny vocabulary, single characters otherwise
    (ids: vocabulary index, or 1000 + code point)."""
    ids, i = [], 0
    while i < len(text):
        best = max((w for w in VOCAB if text.startswith(w, i)), key=len, default=None)
        if best is None:
            ids.append(1000 + ord(text[i]))
            i += 1
        else:
            ids.append(VOCAB.index(best))
            i += len(best)
    return ids


def toy_detokenize(ids):
    return "".join(VOCAB[t] if t < 1000 else chr(t - 1000) for t in ids)


def test_splitmix64_published_vector():
    # first outputs of SplitMix64 seeded with 0 (the reference implementation's well-known sequence)
    assert [fo.splitmix64(0, i) for i in range(3)] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_cuts_cover_the_text_with_lengths_in_range_and_uniform():
    cuts = fo.segment_cuts(7, 2_000_000)
    lens = np.diff([0] + cuts)
    assert cuts[-1] == 2_000_000 and (lens[:-1] >= 1).all() and (lens[:-1] <= 200).all() and 1 <= lens[-1] <= 200
    assert abs(lens[:-1].mean() - 100.5) < 1.0                     # uniform on [1, 200]
    hist = np.bincount(lens[:-1], minlength=201)[1:]
    assert hist.min() > 0 and hist.max() < 2.0 * hist.mean()
    assert fo.segment_cuts(7, 0) == [] and fo.segment_cuts(7, 1) == [1]


def test_fragments_put_subword_pieces_inside_the_text():
    """Fig. 5 / Fig. 9: tokenised whole, `complete` is one token; cut inside it, the pieces
    `comp` + `lete` appear - and the text is still recovered exactly."""
    text = "code complete(models)"
    whole = toy_tokenize(text)
    assert VOCAB.index("complete") in whole
    # a cut after "code comp": segments tokenised separately
    pieces = toy_tokenize(text[:9]) + toy_tokenize(text[9:])
    assert VOCAB.index("comp") in pieces and VOCAB.index("lete") in pieces and VOCAB.index("complete") not in pieces
    assert toy_detokenize(pieces) == text == toy_detokenize(whole)
    rng = np.random.default_rng(0)
    doc = "".join(rng.choice(VOCAB + list("xyz_ ")) for _ in range(3000))
    ids = fo.fragment_tokenize(doc, toy_tokenize, 3, 1, 20)
    assert toy_detokenize(ids) == doc and ids != toy_tokenize(doc)


def test_fim_example_layout():
    doc = "def complete(self):\n    return self.model\n" * 20
    ids = fo.fim_fragment_example(doc, toy_tokenize, 11, 9001, 9002, 9003, 1, 30)
    p, s, m = ids.index(9001), ids.index(9002), ids.index(9003)
    assert p == 0 < s < m and [ids.count(t) for t in (9001, 9002, 9003)] == [1, 1, 1]
    a, b = fo.fim_split(11, len(doc))
    assert 0 <= a <= b <= len(doc)
    assert toy_detokenize(ids[1:s]) == doc[:a] and toy_detokenize(ids[s + 1:m]) == doc[b:] \
        and toy_detokenize(ids[m + 1:]) == doc[a:b]             # PSM order: the middle goes last


@pytest.mark.parametrize("seed,n,lo,hi", [(0, 0, 1, 200), (1, 1, 1, 200), (2, 12345, 1, 200), (2**63 + 5, 99999, 3, 7),
                                          (9, 200, 200, 200)])
def test_library_cuts_equal_oracle(seed, n, lo, hi):
    assert fr.segment_cuts(seed, n, lo, hi).tolist() == fo.segment_cuts(seed, n, lo, hi)
    assert fr.fim_split(seed, n) == fo.fim_split(seed, n)


def test_library_example_equals_oracle_and_rejects_bad_ranges():
    doc = "def complete(self):\n    return self.models\n" * 50
    for seed in range(5):
        assert fr.fim_fragment_example(doc, toy_tokenize, seed, 9001, 9002, 9003) == \
            fo.fim_fragment_example(doc, toy_tokenize, seed, 9001, 9002, 9003)
    from paper_2505_21889_b200 import EfimError
    for bad in [(-1, 1, 200), (10, 0, 200), (10, 5, 4)]:
        with pytest.raises(EfimError):
            fr.segment_cuts(1, *bad)


def test_library_spans_are_the_psm_layout():
    """The span list itself, against facts that need no oracle: markers in the order P, S, M;
    the text spans between them tile prefix [0,a), suffix [b,n), middle [a,b) without gaps;
    every segment but a part's last is within [lo, hi]."""
    n, lo, hi = 5000, 3, 40
    spans = fr.fim_fragment_spans(5, n, lo, hi).tolist()
    a, b = fr.fim_split(5, n)
    kinds = [k for k, _, _ in spans if k != 0]
    assert kinds == [1, 2, 3]
    parts, cur = [], None
    for kind, begin, end in spans:
        if kind != 0:
            cur = []
            parts.append(cur)
            assert begin == end
        else:
            cur.append((begin, end))
    for part, (pb, pe) in zip(parts, [(0, a), (b, n), (a, b)]):
        pos = pb
        for i, (begin, end) in enumerate(part):
            assert begin == pos and end > begin
            assert end - begin <= hi and (i == len(part) - 1 or end - begin >= lo)
            pos = end
        assert pos == pe


def test_command_emits_fragment_tokenised_examples(tmp_path, capsys):
    import json
    doc = "def complete(self):\n    return self.models\n" * 30
    f1, f2 = tmp_path / "a.py", tmp_path / "b.py"
    f1.write_text(doc)
    f2.write_text(doc[::-1])
    assert fr.main([str(f1), str(f2), "--seed", "3", "--hi", "50", "--tokenizer", "chars",
                    "--special", "70001", "70002", "70003"]) == 0
    lines = [json.loads(ln) for ln in capsys.readouterr().out.splitlines()]
    assert [ln["seed"] for ln in lines] == [3, 7] and lines[0]["chars"] == len(doc)
    for ln, text in zip(lines, (doc, doc[::-1])):
        want = fo.fim_fragment_example(text, lambda seg: [ord(c) for c in seg], ln["seed"], 70001, 70002, 70003, 1, 50)
        assert ln["input_ids"] == want
        ids = ln["input_ids"]
        s_at, m_at = ids.index(70002), ids.index(70003)
        back = lambda xs: "".join(chr(t) for t in xs)
        assert back(ids[1:s_at]) + back(ids[m_at + 1:]) + back(ids[s_at + 1:m_at]) == text   # prefix+middle+suffix
    # the default tokenizer: UTF-8 bytes
    assert fr.main([str(f1), "--seed", "1"]) == 0
    out = json.loads(capsys.readouterr().out)
    assert max(out["input_ids"]) <= 258 and out["segments"] >= 3
