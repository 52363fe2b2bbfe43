// Host-side page bookkeeping for a paged KV cache shared by sequences that join and leave between
// steps (the serving setting of Sec. 4.3).  No device code: a free list of pages and one page
// list per slot.  Pages are handed out lowest index first from a stack of free pages, so that a
// test can predict them; nothing else depends on the order.
#include "../../include/space.h"
#include <new>
#include <vector>

struct space_pager {
  int32_t n_pages, pages_per_seq, max_slots;
  std::vector<int32_t> free_pages;                 // stack: back() is handed out next
  std::vector<int32_t> table;                      // [max_slots][pages_per_seq], -1 = no page
  std::vector<int32_t> held;                       // pages a slot holds, -1 = slot not in use
};

namespace {
bool slot_in_use(const space_pager* p, int32_t slot) {
  return slot >= 0 && slot < p->max_slots && p->held[slot] >= 0;
}
}  // namespace

extern "C" {

int space_pager_create(int32_t n_pages, int32_t pages_per_seq, int32_t max_slots, space_pager** out) {
  if (!out || n_pages < 1 || pages_per_seq < 1 || max_slots < 1) return SPACE_E_INVALID_ARG;
  space_pager* p = new (std::nothrow) space_pager;
  if (!p) return SPACE_E_WORKSPACE;
  p->n_pages = n_pages; p->pages_per_seq = pages_per_seq; p->max_slots = max_slots;
  p->free_pages.resize(n_pages);
  for (int32_t i = 0; i < n_pages; ++i) p->free_pages[i] = n_pages - 1 - i;   // page 0 on top
  p->table.assign((size_t)max_slots * pages_per_seq, -1);
  p->held.assign(max_slots, -1);
  *out = p;
  return SPACE_OK;
}

void space_pager_destroy(space_pager* p) { delete p; }

int space_pager_admit(space_pager* p, int32_t* slot) {
  if (!p || !slot) return SPACE_E_INVALID_ARG;
  for (int32_t s = 0; s < p->max_slots; ++s) {
    if (p->held[s] < 0) { p->held[s] = 0; *slot = s; return SPACE_OK; }
  }
  return SPACE_E_WORKSPACE;
}

int space_pager_reserve(space_pager* p, int32_t slot, int32_t n_rows) {
  if (!p || !slot_in_use(p, slot) || n_rows < 0) return SPACE_E_INVALID_ARG;
  const int64_t want = ((int64_t)n_rows + SPACE_PAGE_SIZE - 1) / SPACE_PAGE_SIZE;
  if (want > p->pages_per_seq) return SPACE_E_INVALID_ARG;
  const int32_t have = p->held[slot];
  if (want <= have) return SPACE_OK;                               // pages are given back only by release
  if ((int64_t)p->free_pages.size() < want - have) return SPACE_E_WORKSPACE;
  for (int32_t j = have; j < (int32_t)want; ++j) {
    p->table[(size_t)slot * p->pages_per_seq + j] = p->free_pages.back();
    p->free_pages.pop_back();
  }
  p->held[slot] = (int32_t)want;
  return SPACE_OK;
}

int space_pager_release(space_pager* p, int32_t slot) {
  if (!p || !slot_in_use(p, slot)) return SPACE_E_INVALID_ARG;
  for (int32_t j = p->held[slot] - 1; j >= 0; --j) {
    int32_t& e = p->table[(size_t)slot * p->pages_per_seq + j];
    p->free_pages.push_back(e);
    e = -1;
  }
  p->held[slot] = -1;
  return SPACE_OK;
}

int32_t space_pager_free_pages(const space_pager* p) { return p ? (int32_t)p->free_pages.size() : -1; }

int32_t space_pager_rows(const space_pager* p, int32_t slot) {
  if (!p || !slot_in_use(p, slot)) return -1;
  return p->held[slot] * SPACE_PAGE_SIZE;
}

int space_pager_batch_table(const space_pager* p, const int32_t* slots, int32_t n, int32_t* table_out) {
  if (!p || n < 0 || (n > 0 && (!slots || !table_out))) return SPACE_E_INVALID_ARG;
  for (int32_t i = 0; i < n; ++i)
    if (!slot_in_use(p, slots[i])) return SPACE_E_INVALID_ARG;
  for (int32_t i = 0; i < n; ++i)
    for (int32_t j = 0; j < p->pages_per_seq; ++j)
      table_out[(size_t)i * p->pages_per_seq + j] = p->table[(size_t)slots[i] * p->pages_per_seq + j];
  return SPACE_OK;
}

}  // extern "C"
