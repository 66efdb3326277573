// Host-side EFIM front end: the prompt transformation of Sec. 3.1 (steps 1-5) and the
// page-granular cross-request KV reuse (Sec. 1) that produce cached_len / block tables
// for the GPU calls.  Plain C++; compiled with the kernels so that one library holds
// the whole path.  No CUDA call is made here.
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <set>
#include <unordered_map>
#include <vector>
#include "efim.h"

namespace {

struct Session {
  std::vector<int32_t> prefix, suffix;     // as laid out in the user's last prompt
};

// A cached page: the block of tokens it holds and the page holding the block before it.
// (parent, tokens) names the whole token prefix: a parent is evicted only after all its
// children (it is never older than they are, and among equals the deeper page goes first),
// so a parent id in a live key always means the same chain.
struct PageKey {
  int32_t parent;
  std::vector<int32_t> tokens;
  bool operator==(const PageKey& o) const { return parent == o.parent && tokens == o.tokens; }
};
struct PageKeyHash {
  size_t operator()(const PageKey& k) const {
    uint64_t h = 0x9e3779b97f4a7c15ull ^ (uint64_t)(uint32_t)k.parent;
    for (int32_t t : k.tokens) {
      h ^= (uint64_t)(uint32_t)t + 0x9e3779b97f4a7c15ull + (h << 6) + (h >> 2);
    }
    return (size_t)h;
  }
};
struct PageMeta {
  bool cached = false;
  int32_t ref = 0, depth = 0;
  int64_t used = 0;
  PageKey key;
};
struct Request {
  int32_t n_matched;
  std::vector<int32_t> pages;
};

}  // namespace

struct efim_frontend {
  int32_t tok_p, tok_s, tok_m, rebase, page_size;
  std::unordered_map<int64_t, Session> sessions;
  std::set<int32_t> free_pages;
  std::vector<PageMeta> pages;
  std::unordered_map<PageKey, int32_t, PageKeyHash> by_key;
  // unpinned cached pages in eviction order: oldest use first, deepest first among equals
  std::set<std::tuple<int64_t, int32_t, int32_t>> evictable;
  std::unordered_map<int64_t, Request> requests;
  int64_t tick = 0, next_handle = 1, prompt_tokens = 0, hit_tokens = 0, evictions = 0;

  std::tuple<int64_t, int32_t, int32_t> order_of(int32_t pid) const {
    return std::make_tuple(pages[pid].used, -pages[pid].depth, pid);
  }
  void touch(int32_t pid) {                 // new use time; keeps the eviction order current
    PageMeta& m = pages[pid];
    if (m.cached && m.ref == 0) evictable.erase(order_of(pid));
    m.used = tick;
    if (m.cached && m.ref == 0) evictable.insert(order_of(pid));
  }
  void pin(int32_t pid) {
    PageMeta& m = pages[pid];
    if (m.ref == 0) evictable.erase(order_of(pid));
    ++m.ref;
  }
  void unpin(int32_t pid) {
    PageMeta& m = pages[pid];
    if (--m.ref == 0) evictable.insert(order_of(pid));
  }
  int32_t take_page() {
    if (!free_pages.empty()) {
      const int32_t pid = *free_pages.begin();
      free_pages.erase(free_pages.begin());
      return pid;
    }
    if (evictable.empty()) return -1;
    const int32_t pid = std::get<2>(*evictable.begin());
    evictable.erase(evictable.begin());
    by_key.erase(pages[pid].key);
    pages[pid] = PageMeta{};
    ++evictions;
    return pid;
  }
};

extern "C" efim_frontend* efim_frontend_create(int32_t tok_p, int32_t tok_s, int32_t tok_m, int32_t rebase_inc_tokens,
                                               int32_t num_pages, int32_t page_size) {
  if (num_pages <= 0 || page_size <= 0) return nullptr;
  efim_frontend* fe = new efim_frontend();
  fe->tok_p = tok_p; fe->tok_s = tok_s; fe->tok_m = tok_m;
  fe->rebase = rebase_inc_tokens; fe->page_size = page_size;
  fe->pages.resize((size_t)num_pages);
  for (int32_t i = 0; i < num_pages; ++i) fe->free_pages.insert(fe->free_pages.end(), i);
  return fe;
}

extern "C" void efim_frontend_destroy(efim_frontend* fe) { delete fe; }

extern "C" efim_status efim_frontend_transform(efim_frontend* fe, int64_t user, const int32_t* h_prefix,
                                               int32_t prefix_len, const int32_t* h_suffix, int32_t suffix_len,
                                               int32_t* h_prompt, int32_t capacity, int32_t* prompt_len,
                                               int32_t* format, int32_t* inc_len) {
  if (!fe || prefix_len < 0 || suffix_len < 0 || (prefix_len && !h_prefix) || (suffix_len && !h_suffix) ||
      !h_prompt || !prompt_len || !format || !inc_len)
    return EFIM_ERR_INVALID_ARG;
  if ((int64_t)capacity < (int64_t)prefix_len + suffix_len + 3) return EFIM_ERR_OUT_OF_RANGE;
  const std::vector<int32_t> prefix(h_prefix, h_prefix + prefix_len), suffix(h_suffix, h_suffix + suffix_len);
  int32_t fmt, common = prefix_len;                        // tokens of the prefix placed before <S>
  auto it = fe->sessions.find(user);                       // step 1
  if (it == fe->sessions.end()) {                          // step 2
    fe->sessions[user] = Session{prefix, suffix};
    fmt = EFIM_FMT_PSM_NEW;
  } else {                                                 // step 3
    Session& s = it->second;
    const int32_t base = (int32_t)s.prefix.size();
    const bool extends = prefix_len >= base && std::equal(s.prefix.begin(), s.prefix.end(), prefix.begin());
    if (extends && prefix_len > base) {                    // step 4
      if (fe->rebase > 0 && prefix_len - base > fe->rebase) {
        s = Session{prefix, suffix};
        fmt = EFIM_FMT_PSM_REBASE;
      } else {
        s.suffix = suffix;
        common = base;
        fmt = EFIM_FMT_EFIM;
      }
    } else if (extends) {                                  // step 5, or the same request again
      fmt = suffix == s.suffix ? EFIM_FMT_PSM_SAME : EFIM_FMT_PSM_SUFFIX;
      s.suffix = suffix;
    } else {                                               // prefix edited: start over
      s = Session{prefix, suffix};
      fmt = EFIM_FMT_PSM_RESET;
    }
  }
  int32_t n = 0;
  h_prompt[n++] = fe->tok_p;
  for (int32_t i = 0; i < common; ++i) h_prompt[n++] = prefix[i];
  h_prompt[n++] = fe->tok_s;
  for (int32_t i = 0; i < suffix_len; ++i) h_prompt[n++] = suffix[i];
  h_prompt[n++] = fe->tok_m;
  for (int32_t i = common; i < prefix_len; ++i) h_prompt[n++] = prefix[i];   // inc goes last (Sec. 1)
  *prompt_len = n;
  *format = fmt;
  *inc_len = prefix_len - common;
  return EFIM_OK;
}

extern "C" efim_status efim_frontend_admit(efim_frontend* fe, const int32_t* h_prompt, int32_t prompt_len,
                                           int32_t reserve_tokens, int32_t* h_block_table_row,
                                           int32_t max_pages_per_seq, int32_t* cached_len, int32_t* num_pages_out,
                                           int64_t* handle) {
  if (!fe || !h_prompt || prompt_len <= 0 || reserve_tokens < 0 || !h_block_table_row || max_pages_per_seq <= 0 ||
      !cached_len || !num_pages_out || !handle)
    return EFIM_ERR_INVALID_ARG;
  const int32_t P = fe->page_size;
  const int64_t total_pages = ((int64_t)prompt_len + reserve_tokens + P - 1) / P;
  if (total_pages > max_pages_per_seq) return EFIM_ERR_OUT_OF_RANGE;
  ++fe->tick;
  Request rq;
  int32_t parent = -1;
  for (int32_t b = 0; b < prompt_len / P; ++b) {
    PageKey key{parent, std::vector<int32_t>(h_prompt + (size_t)b * P, h_prompt + (size_t)(b + 1) * P)};
    auto it = fe->by_key.find(key);
    if (it == fe->by_key.end()) break;
    parent = it->second;
    rq.pages.push_back(parent);
  }
  if (!rq.pages.empty() && (int64_t)rq.pages.size() * P >= prompt_len) rq.pages.pop_back();   // one token is computed
  rq.n_matched = (int32_t)rq.pages.size();
  for (int32_t pid : rq.pages) {
    fe->pin(pid);
    fe->pages[pid].used = fe->tick;
  }
  for (int64_t i = rq.n_matched; i < total_pages; ++i) {
    const int32_t pid = fe->take_page();
    if (pid < 0) {                                         // nothing left to take: undo
      for (size_t k = rq.n_matched; k < rq.pages.size(); ++k) {
        fe->pages[rq.pages[k]] = PageMeta{};
        fe->free_pages.insert(rq.pages[k]);
      }
      for (int32_t k = 0; k < rq.n_matched; ++k) fe->unpin(rq.pages[k]);
      return EFIM_ERR_WORKSPACE;
    }
    fe->pages[pid].ref = 1;
    rq.pages.push_back(pid);
  }
  for (int32_t i = 0; i < max_pages_per_seq; ++i)
    h_block_table_row[i] = i < (int32_t)rq.pages.size() ? rq.pages[i] : -1;
  *cached_len = rq.n_matched * P;
  *num_pages_out = (int32_t)rq.pages.size();
  *handle = fe->next_handle++;
  fe->prompt_tokens += prompt_len;
  fe->hit_tokens += (int64_t)rq.n_matched * P;
  fe->requests[*handle] = std::move(rq);
  return EFIM_OK;
}

extern "C" efim_status efim_frontend_finish(efim_frontend* fe, int64_t handle, const int32_t* h_tokens,
                                            int32_t total_len) {
  if (!fe || total_len < 0 || (total_len && !h_tokens)) return EFIM_ERR_INVALID_ARG;
  auto rit = fe->requests.find(handle);
  if (rit == fe->requests.end()) return EFIM_ERR_INVALID_ARG;
  const Request rq = std::move(rit->second);
  fe->requests.erase(rit);
  const int32_t P = fe->page_size;
  ++fe->tick;
  int32_t parent = -1;
  for (int32_t b = 0; b < (int32_t)rq.pages.size(); ++b) {
    const int32_t pid = rq.pages[b];
    if (b < rq.n_matched) {
      fe->pages[pid].used = fe->tick;
      fe->unpin(pid);
      parent = pid;
    } else if ((int64_t)(b + 1) * P <= total_len) {
      PageKey key{parent, std::vector<int32_t>(h_tokens + (size_t)b * P, h_tokens + (size_t)(b + 1) * P)};
      auto it = fe->by_key.find(key);
      if (it != fe->by_key.end()) {                        // the same content was registered meanwhile
        fe->touch(it->second);
        parent = it->second;
        fe->pages[pid] = PageMeta{};
        fe->free_pages.insert(pid);
      } else {
        PageMeta& m = fe->pages[pid];
        m.cached = true; m.ref = 0; m.depth = b + 1; m.used = fe->tick; m.key = key;
        fe->by_key.emplace(std::move(key), pid);
        fe->evictable.insert(fe->order_of(pid));
        parent = pid;
      }
    } else {
      fe->pages[pid] = PageMeta{};
      fe->free_pages.insert(pid);
    }
  }
  return EFIM_OK;
}

extern "C" void efim_frontend_stats(const efim_frontend* fe, int64_t* h_out) {
  if (!fe || !h_out) return;
  h_out[0] = fe->prompt_tokens;
  h_out[1] = fe->hit_tokens;
  h_out[2] = fe->evictions;
  h_out[3] = (int64_t)fe->free_pages.size();
}
