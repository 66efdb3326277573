// Fragment tokenisation, Sec. 3.2: where a text is cut into the segments that are then
// tokenised one by one.  Host code only (the tokenizer is the caller's); compiled into
// the library so that training-data tools and the serving path share one binary.
#include <cstdint>
#include "efim.h"

namespace {
// SplitMix64 (Steele, Lea, Flood 2014), used as a counter-based generator: draw i of a seed
inline uint64_t splitmix64(uint64_t seed, uint64_t i) {
  uint64_t z = seed + (i + 1) * 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
}  // namespace

extern "C" int64_t efim_fragment_cuts(uint64_t seed, int64_t n, int32_t lo, int32_t hi, int64_t* h_cuts,
                                      int64_t capacity) {
  if (n < 0 || lo < 1 || hi < lo || capacity < 0 || (capacity > 0 && !h_cuts)) return -1;
  const uint64_t span = (uint64_t)(hi - lo) + 1;
  int64_t pos = 0, count = 0;
  for (uint64_t i = 0; pos < n; ++i) {
    const int64_t len = lo + (int64_t)(splitmix64(seed, i) % span);
    pos = (n - pos <= len) ? n : pos + len;
    if (count < capacity) h_cuts[count] = pos;
    ++count;
  }
  return count;
}

extern "C" efim_status efim_fim_split(uint64_t seed, int64_t n, int64_t* a, int64_t* b) {
  if (n < 0 || !a || !b) return EFIM_ERR_INVALID_ARG;
  const uint64_t s = seed ^ 0x46494D5F53504C54ull;
  int64_t x = (int64_t)(splitmix64(s, 0) % (uint64_t)(n + 1)), y = (int64_t)(splitmix64(s, 1) % (uint64_t)(n + 1));
  if (x > y) { const int64_t t = x; x = y; y = t; }
  *a = x;
  *b = y;
  return EFIM_OK;
}

// The spans of one training example, in emission order.  A text span is one segment of one of
// the three parts; the special tokens sit between the parts: <P> prefix.. <S> suffix.. <M> middle..
extern "C" int64_t efim_fim_fragment_spans(uint64_t seed, int64_t n, int32_t lo, int32_t hi, int64_t* h_spans,
                                           int64_t capacity) {
  if (n < 0 || lo < 1 || hi < lo || capacity < 0 || (capacity > 0 && !h_spans)) return -1;
  int64_t a = 0, b = 0;
  if (efim_fim_split(seed, n, &a, &b) != EFIM_OK) return -1;
  const uint64_t span = (uint64_t)(hi - lo) + 1;
  int64_t count = 0;
  auto emit = [&](int64_t kind, int64_t begin, int64_t end) {
    if (count < capacity) {
      h_spans[3 * count] = kind;
      h_spans[3 * count + 1] = begin;
      h_spans[3 * count + 2] = end;
    }
    ++count;
  };
  // part k is segmented with the generator under seed + 1 + k (prefix, suffix, middle)
  const int64_t part_begin[3] = {0, b, a}, part_end[3] = {a, n, b};
  const int64_t marker[3] = {EFIM_SPAN_TOKEN_P, EFIM_SPAN_TOKEN_S, EFIM_SPAN_TOKEN_M};
  for (int k = 0; k < 3; ++k) {
    emit(marker[k], part_begin[k], part_begin[k]);
    int64_t pos = part_begin[k];
    for (uint64_t i = 0; pos < part_end[k]; ++i) {
      const int64_t len = lo + (int64_t)(splitmix64(seed + 1 + (uint64_t)k, i) % span);
      const int64_t next = (part_end[k] - pos <= len) ? part_end[k] : pos + len;
      emit(EFIM_SPAN_TEXT, pos, next);
      pos = next;
    }
  }
  return count;
}
