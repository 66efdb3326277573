"""CPU oracle for the fragment-tokenisation data processing of Sec. 3.2 (Fig. 8, Fig. 9).

TEST INFRASTRUCTURE ONLY; shares no code with the library.

The paper: FIM training data is a document cut into prefix / middle / suffix, reordered
(PSM: `<P>prefix<S>suffix<M>middle`) and tokenised part by part; fragment tokenisation
cuts the text further into segments whose lengths are uniform in [1, 200] and tokenises
every segment on its own, so that sub-word pieces appear everywhere and not only next to
the special tokens.  Readings (the paper's figures are lost): a segment's length counts
characters; each of the three parts is segmented on its own (a segment never spans a
special token); the last segment of a part is whatever is left.

Random numbers: the method draws them, so oracle and library both implement one
counter-based generator from its published definition - SplitMix64 (Steele, Lea, Flood
2014): z = seed + (i + 1) * 0x9E3779B97F4A7C15, two xor-shift-multiply rounds, final
xor-shift - and the i-th length is lo + z_i mod (hi - lo + 1).

Parity unpinned against the paper (it prints no example with numbers).
"""
MASK = (1 << 64) - 1


def splitmix64(seed, i):
    z = (seed + (i + 1) * 0x9E3779B97F4A7C15) & MASK
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK
    return z ^ (z >> 31)


def segment_cuts(seed, n, lo=1, hi=200):
    """End offsets of the segments of a text of n characters (the last one is n)."""
    cuts, pos, i = [], 0, 0
    while pos < n:
        pos = min(n, pos + lo + splitmix64(seed, i) % (hi - lo + 1))
        cuts.append(pos)
        i += 1
    return cuts


def fragment_tokenize(text, tokenize, seed, lo=1, hi=200):
    """Token ids of the text, every segment tokenised on its own (Sec. 3.2)."""
    ids, start = [], 0
    for end in segment_cuts(seed, len(text), lo, hi):
        ids.extend(tokenize(text[start:end]))
        start = end
    return ids


def fim_split(seed, n):
    """Two cut points 0 <= a <= b <= n of a document of n characters: prefix [0,a),
    middle [a,b), suffix [b,n) (draws 0 and 1 of the generator under seed ^ FIM_SALT)."""
    s = seed ^ 0x46494D5F53504C54
    a, b = splitmix64(s, 0) % (n + 1), splitmix64(s, 1) % (n + 1)
    return (a, b) if a <= b else (b, a)


def fim_fragment_example(text, tokenize, seed, tok_p, tok_s, tok_m, lo=1, hi=200):
    """`<P>prefix<S>suffix<M>middle` with each part fragment-tokenised (seeds seed+1, +2, +3)."""
    a, b = fim_split(seed, len(text))
    prefix, middle, suffix = text[:a], text[a:b], text[b:]
    return ([tok_p] + fragment_tokenize(prefix, tokenize, seed + 1, lo, hi) +
            [tok_s] + fragment_tokenize(suffix, tokenize, seed + 2, lo, hi) +
            [tok_m] + fragment_tokenize(middle, tokenize, seed + 3, lo, hi))
