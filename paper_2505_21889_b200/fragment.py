"""Fragment tokenisation (Sec. 3.2): cut a text into segments whose lengths are uniform
in [1, 200] characters, tokenise every segment on its own, concatenate.  The cut points
come from the library (efim_fragment_cuts, efim_fim_split); the tokenizer is any callable
`str -> list[int]` of the caller's."""
import ctypes

import numpy as np

from .binding import load_library, EfimError


def _lib():
    lib = load_library()
    lib.efim_fragment_cuts.restype = ctypes.c_int64
    lib.efim_fragment_cuts.argtypes = [ctypes.c_uint64, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32,
                                       ctypes.c_void_p, ctypes.c_int64]
    lib.efim_fim_split.restype = ctypes.c_int
    lib.efim_fim_split.argtypes = [ctypes.c_uint64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
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
    ids, start = [], 0
    for end in segment_cuts(seed, len(text), lo, hi).tolist():
        ids.extend(tokenize(text[start:end]))
        start = end
    return ids


def fim_split(seed, n):
    a, b = ctypes.c_int64(), ctypes.c_int64()
    st = _lib().efim_fim_split(seed, n, ctypes.addressof(a), ctypes.addressof(b))
    if st != 0:
        raise EfimError(st, "efim_fim_split")
    return a.value, b.value


def fim_fragment_example(text, tokenize, seed, tok_p, tok_s, tok_m, lo=1, hi=200):
    """One training example: `<P>prefix<S>suffix<M>middle`, each part fragment-tokenised."""
    a, b = fim_split(seed, len(text))
    return ([tok_p] + fragment_tokenize(text[:a], tokenize, seed + 1, lo, hi) +
            [tok_s] + fragment_tokenize(text[b:], tokenize, seed + 2, lo, hi) +
            [tok_m] + fragment_tokenize(text[a:b], tokenize, seed + 3, lo, hi))
