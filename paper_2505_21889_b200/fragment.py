"""Fragment tokenisation (Sec. 3.2): a text is cut into segments whose lengths are uniform
in [1, 200] characters and every segment is tokenised on its own.  Where the cuts fall, and
how a FIM training example is laid out, is decided by the library (efim_fragment_cuts,
efim_fim_fragment_spans); this module applies the caller's tokenizer - any callable
`str -> list[int]` - to the spans it is given.

As a command it turns text files into fragment-tokenised FIM examples, one JSON line each:

    python -m paper_2505_21889_b200.fragment FILE [FILE ...] --seed 7 [--lo 1 --hi 200]
        [--tokenizer bytes | chars | package.module:callable] [--special 256 257 258]

`bytes` (the default) maps a segment to its UTF-8 bytes, `chars` to its code points; a
`module:callable` is imported and called with each segment.
"""
import ctypes
import importlib
import json
import sys

import numpy as np

from .binding import load_library, EfimError

SPAN_TEXT = 0


def _lib():
    lib = load_library()
    lib.efim_fragment_cuts.restype = ctypes.c_int64
    lib.efim_fragment_cuts.argtypes = [ctypes.c_uint64, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32,
                                       ctypes.c_void_p, ctypes.c_int64]
    lib.efim_fim_split.restype = ctypes.c_int
    lib.efim_fim_split.argtypes = [ctypes.c_uint64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
    lib.efim_fim_fragment_spans.restype = ctypes.c_int64
    lib.efim_fim_fragment_spans.argtypes = [ctypes.c_uint64, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32,
                                            ctypes.c_void_p, ctypes.c_int64]
    return lib


def segment_cuts(seed, n, lo=1, hi=200) -> np.ndarray:
    """End offsets of the segments of a text of n characters (int64; the last one is n)."""
    lib = _lib()
    count = lib.efim_fragment_cuts(seed, n, lo, hi, None, 0)
    if count < 0:
        raise EfimError(1, "efim_fragment_cuts")
    cuts = np.empty(count, np.int64)
    lib.efim_fragment_cuts(seed, n, lo, hi, cuts.ctypes.data, count)
    return cuts


def fragment_tokenize(text, tokenize, seed, lo=1, hi=200):
    """Token ids of `text`, each of the library's segments tokenised separately."""
    ends = segment_cuts(seed, len(text), lo, hi)
    begins = np.concatenate([np.zeros(1, np.int64), ends[:-1]])
    return [t for b, e in zip(begins.tolist(), ends.tolist()) for t in tokenize(text[b:e])]


def fim_split(seed, n):
    a, b = ctypes.c_int64(), ctypes.c_int64()
    st = _lib().efim_fim_split(seed, n, ctypes.addressof(a), ctypes.addressof(b))
    if st != 0:
        raise EfimError(st, "efim_fim_split")
    return a.value, b.value


def fim_fragment_spans(seed, n, lo=1, hi=200) -> np.ndarray:
    """The example's spans as the library lays them out: int64 [count, 3] of (kind, begin, end)."""
    lib = _lib()
    count = lib.efim_fim_fragment_spans(seed, n, lo, hi, None, 0)
    if count < 0:
        raise EfimError(1, "efim_fim_fragment_spans")
    spans = np.empty((count, 3), np.int64)
    lib.efim_fim_fragment_spans(seed, n, lo, hi, spans.ctypes.data, count)
    return spans


def fim_fragment_example(text, tokenize, seed, tok_p, tok_s, tok_m, lo=1, hi=200):
    """One training example: the library's spans, text spans through `tokenize`, the three
    marker kinds replaced by the caller's special-token ids."""
    special = {1: tok_p, 2: tok_s, 3: tok_m}
    ids = []
    for kind, begin, end in fim_fragment_spans(seed, len(text), lo, hi).tolist():
        if kind == SPAN_TEXT:
            ids += tokenize(text[begin:end])
        else:
            ids.append(special[kind])
    return ids


def _resolve_tokenizer(spec):
    if spec == "bytes":
        return lambda seg: list(seg.encode("utf-8"))
    if spec == "chars":
        return lambda seg: [ord(ch) for ch in seg]
    module, _, name = spec.partition(":")
    if not name:
        raise SystemExit(f"--tokenizer {spec!r}: expected bytes, chars or package.module:callable")
    return getattr(importlib.import_module(module), name)


def main(argv=None):
    import argparse
    ap = argparse.ArgumentParser(prog="python -m paper_2505_21889_b200.fragment", description=__doc__.split("\n\n")[0])
    ap.add_argument("files", nargs="+", help="text files; each is one document")
    ap.add_argument("--seed", type=int, default=0, help="document i uses seed + 4*i")
    ap.add_argument("--lo", type=int, default=1)
    ap.add_argument("--hi", type=int, default=200)
    ap.add_argument("--tokenizer", default="bytes")
    ap.add_argument("--special", type=int, nargs=3, default=[256, 257, 258], metavar=("P", "S", "M"))
    args = ap.parse_args(argv)
    tokenize = _resolve_tokenizer(args.tokenizer)
    for i, path in enumerate(args.files):
        with open(path, encoding="utf-8") as f:
            text = f.read()
        seed = args.seed + 4 * i                  # an example uses seed .. seed+3
        ids = fim_fragment_example(text, tokenize, seed, *args.special, lo=args.lo, hi=args.hi)
        a, b = fim_split(seed, len(text))
        print(json.dumps({"file": path, "seed": seed, "chars": len(text), "prefix_end": a, "middle_end": b,
                          "segments": int((fim_fragment_spans(seed, len(text), args.lo, args.hi)[:, 0] == 0).sum()),
                          "input_ids": [int(t) for t in ids]}))
    return 0


if __name__ == "__main__":
    sys.exit(main())
