// Index checks of the paged cache and the GEMM workspace, written once for the host and the device.
// The kernels call them when the library is built with -DCORUN_CHECKED (a failed check records DEV_BAD_INDEX
// in the status word and the access is skipped or redirected to the reserved page 0: nothing faults); the
// unit tests call the same functions on the host through corun_debug_check_index.
#pragma once
#include <stdint.h>

#ifndef __CUDACC__
#define CORUN_HD
#else
#define CORUN_HD __host__ __device__
#endif

namespace corun {

// A row of the program may use (slot, position pos) when the slot exists and the position lies inside the
// block table's reach.
CORUN_HD inline bool check_slot_pos(long long slot, long long n_slots, long long pos, long long max_blocks, long long kv_block) {
  return slot >= 0 && slot < n_slots && pos >= 0 && kv_block > 0 && pos / kv_block < max_blocks;
}
// A page number read from a block table must name a page of the pool.
CORUN_HD inline bool check_page(long long page, long long pool_blocks) { return page >= 0 && page < pool_blocks; }
// An attention item (row, kv head, split) must lie inside the program's shape and the row's own context.
CORUN_HD inline bool check_item(long long row, long long n_rows, long long head, long long n_kv, long long split, long long ctx,
                                long long split_tokens) {
  return row >= 0 && row < n_rows && head >= 0 && head < n_kv && split >= 0 && split_tokens > 0 && split * split_tokens < ctx;
}
// A partial-sum slot (cta, 0 / 1) of the GEMM workspace must exist.
CORUN_HD inline bool check_ws_slot(long long cta, long long slot, long long grid) { return cta >= 0 && cta < grid && (slot == 0 || slot == 1); }

}  // namespace corun
