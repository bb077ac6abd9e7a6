// Host-side planning for the mixed-batch multi-LoRA layer: segment table -> validated routing
// and the work lists the kernels consume.  Pure C++ (no CUDA), so it can be exercised without a
// GPU through the C ABI (mlora_plan_create with a null context).
#pragma once

#include <cstdint>
#include <vector>

#include "mlora.h"

namespace mlora {

constexpr int kTileRows = 128;     // rows per tensor-core tile of the one-SM kernel (UMMA M = 128)
constexpr int kPairTileRows = 256; // rows per tile of the two-SM kernel (a CTA pair, UMMA M = 256)
constexpr int kItemRows = 32;      // most rows in one shrink work item (two mma.sync row blocks)
constexpr int kItemDescInts = 8;  // ints per packed item record (RowSpace::item_desc)
constexpr int kChunkRows = 16;     // rows per gradient chunk (one mma.sync contraction step)
constexpr int kMaxRank = 128;

// Tables over one row space: the batch rows (forward) or the compact fine-tuning rows (backward).
struct RowSpace {
  int32_t n_rows = 0;
  std::vector<int32_t> row_adapter;    // [n_rows] adapter id or -1
  std::vector<int32_t> row_save;       // [n_rows] save offset of the row or -1 (forward space only)
  // Tensor-core tiles of kTileRows rows: the distinct adapters of a tile ("groups", in order of
  // first appearance) and, per row, the index of its group inside its tile (-1: base only).
  std::vector<int32_t> row_grp;        // [n_rows]
  std::vector<int32_t> tile_grp_off;   // [n_tiles + 1]
  std::vector<int32_t> grp_adapter;    // [tile_grp_off.back()]
  // the same three tables for tiles of kPairTileRows rows
  std::vector<int32_t> row_grp2, tile2_grp_off, grp2_adapter;
  std::vector<int32_t> zero_rows2;     // rows without an adapter inside 256-row tiles that have groups
  // Shrink items: the rows that have an adapter, gathered BY ADAPTER (ascending adapter id, rows
  // ascending inside an adapter) and cut into items of <= kItemRows rows.  Rows of an item need
  // not be adjacent in the batch: decode rows that share an adapter are processed together, so an
  // adapter's matrix is fetched once per item instead of once per row.
  std::vector<int32_t> item_rows;      // [rows with an adapter] row ids, grouped by adapter
  std::vector<int32_t> item_save;      // parallel to item_rows: save offset of that row or -1
  std::vector<int32_t> item_start, item_nrows, item_adapter;
  // One packed record per item for the streaming kernels, kItemDescInts ints:
  // {start, nrows, adapter, flags, first row, first save offset (-1: none), 0, 0}; flag bit 0: the
  // item's rows are consecutive rows of the batch; bit 1: additionally the item is full
  // (kItemRows rows) and its save offsets are consecutive, so its rows can be saved as one block.
  std::vector<int32_t> item_desc;
  // Blocks for the tensor-core shrink: runs of <= kTileRows consecutive rows that share one adapter.
  std::vector<int32_t> tcb_row0, tcb_nrows, tcb_adapter;
  // Plans made with per-adapter ranks only (empty otherwise): in the block-diagonal low-rank operand of a
  // 256-row tile a group is as wide as its adapter's rank rounded up to 16 columns, not as wide as the layer's
  // padded rank.  grp2_col / grp2_width: first column and width of each group; tile2_cols: columns of each
  // tile's operand; the operand's rows on the B side are 16-row PIECES of the adapters' matrices, listed per
  // tile in column order: piece_src = adapter << 8 | (first row of the piece inside the adapter / 16).
  std::vector<int32_t> grp2_col, grp2_width, tile2_cols, tile2_piece_off, piece_src;
  std::vector<int32_t> tcb_width;      // [blocks] rows of the adapter's matrix a block of the tensor-core shrink reads: its rank rounded up to 16, 32, 64 or 128
  int32_t n_tiles() const { return (n_rows + kTileRows - 1) / kTileRows; }
  int32_t n_items() const { return (int32_t)item_start.size(); }
};

struct HostPlan {
  int32_t n_rows = 0, n_adapters = 0, n_segs = 0;
  std::vector<int32_t> adapter_rank;   // [n_adapters] own rank of each adapter, or empty: every adapter has the layer's rank
  int32_t ft_rows = 0;
  std::vector<int32_t> seg_save_off;   // [n_segs] save offset or -1
  std::vector<int32_t> ft_adapters;    // slot -> adapter id
  RowSpace fwd;                        // batch rows
  RowSpace bwd;                        // compact fine-tuning rows, in save order
  // Gradient work: per slot, chunks of <= kChunkRows compact rows.
  std::vector<int32_t> slot_chunk_off; // [n_slots + 1]
  std::vector<int32_t> chunk_row0, chunk_nrows;
  // The same rows as blocks of <= kTileRows consecutive compact rows (tiles of the streaming kernel).
  std::vector<int32_t> slot_blk_off;   // [n_slots + 1]
  std::vector<int32_t> blk_row0, blk_nrows;
  std::vector<int32_t> slot_width;     // ranked plans only: rows of the slot's gradient that exist (its adapter's rank rounded up to 16, 32, 64 or 128)
};

inline void build_tile_groups(const std::vector<int32_t>& row_adapter, int32_t tile_rows,
                              std::vector<int32_t>& row_grp, std::vector<int32_t>& tile_grp_off,
                              std::vector<int32_t>& grp_adapter) {
  const int32_t n = (int32_t)row_adapter.size();
  row_grp.assign(n, -1);
  tile_grp_off.assign(1, 0);
  grp_adapter.clear();
  for (int32_t t0 = 0; t0 < n; t0 += tile_rows) {
    const int32_t t1 = t0 + tile_rows < n ? t0 + tile_rows : n;
    const int32_t base = (int32_t)grp_adapter.size();
    for (int32_t t = t0; t < t1; ++t) {
      const int32_t a = row_adapter[t];
      if (a < 0) continue;
      int32_t g = -1;
      for (int32_t i = base; i < (int32_t)grp_adapter.size(); ++i)
        if (grp_adapter[i] == a) { g = i - base; break; }
      if (g < 0) { g = (int32_t)grp_adapter.size() - base; grp_adapter.push_back(a); }
      row_grp[t] = g;
    }
    tile_grp_off.push_back((int32_t)grp_adapter.size());
  }
}

// Group widths and B-side pieces of a ranked plan (see RowSpace).
inline void build_ranked(RowSpace& rs, const std::vector<int32_t>& adapter_rank) {
  rs.grp2_col.clear(); rs.grp2_width.clear(); rs.tile2_cols.clear(); rs.piece_src.clear();
  rs.tile2_piece_off.assign(1, 0);
  rs.tcb_width.clear();
  for (int32_t a : rs.tcb_adapter) {
    int32_t w = 16;
    while (w < adapter_rank[a]) w *= 2;
    rs.tcb_width.push_back(w);
  }
  for (size_t t = 0; t + 1 < rs.tile2_grp_off.size(); ++t) {
    int32_t col = 0;
    for (int32_t i = rs.tile2_grp_off[t]; i < rs.tile2_grp_off[t + 1]; ++i) {
      const int32_t a = rs.grp2_adapter[i];
      const int32_t w = (adapter_rank[a] + 15) / 16 * 16;
      rs.grp2_col.push_back(col);
      rs.grp2_width.push_back(w);
      for (int32_t j = 0; j < w / 16; ++j) rs.piece_src.push_back((a << 8) | j);
      col += w;
    }
    rs.tile2_cols.push_back(col);
    rs.tile2_piece_off.push_back((int32_t)rs.piece_src.size());
  }
}

inline void build_tiles_and_items(RowSpace& rs) {
  const int32_t n = rs.n_rows;
  build_tile_groups(rs.row_adapter, kTileRows, rs.row_grp, rs.tile_grp_off, rs.grp_adapter);
  build_tile_groups(rs.row_adapter, kPairTileRows, rs.row_grp2, rs.tile2_grp_off, rs.grp2_adapter);
  rs.zero_rows2.clear();
  for (int32_t t = 0; t < n; ++t) {
    const int32_t tile = t / kPairTileRows;
    if (rs.row_adapter[t] < 0 && rs.tile2_grp_off[tile + 1] > rs.tile2_grp_off[tile]) rs.zero_rows2.push_back(t);
  }
  rs.tcb_row0.clear(); rs.tcb_nrows.clear(); rs.tcb_adapter.clear();
  for (int32_t t = 0; t < n; ++t) {
    const int32_t a = rs.row_adapter[t];
    if (a < 0) continue;
    if (!rs.tcb_row0.empty() && rs.tcb_adapter.back() == a && rs.tcb_row0.back() + rs.tcb_nrows.back() == t &&
        rs.tcb_nrows.back() < kTileRows) {
      rs.tcb_nrows.back()++;
    } else {
      rs.tcb_row0.push_back(t); rs.tcb_nrows.push_back(1); rs.tcb_adapter.push_back(a);
    }
  }
  rs.item_rows.clear(); rs.item_start.clear(); rs.item_nrows.clear(); rs.item_adapter.clear(); rs.item_desc.clear();
  int32_t max_adapter = -1;
  for (int32_t t = 0; t < n; ++t) max_adapter = rs.row_adapter[t] > max_adapter ? rs.row_adapter[t] : max_adapter;
  std::vector<int32_t> count(max_adapter + 2, 0);
  for (int32_t t = 0; t < n; ++t) if (rs.row_adapter[t] >= 0) count[rs.row_adapter[t] + 1]++;
  for (int32_t a = 0; a <= max_adapter; ++a) count[a + 1] += count[a];
  rs.item_rows.assign(max_adapter >= 0 ? count[max_adapter + 1] : 0, 0);
  {
    std::vector<int32_t> fill(count.begin(), count.end());
    for (int32_t t = 0; t < n; ++t) if (rs.row_adapter[t] >= 0) rs.item_rows[fill[rs.row_adapter[t]]++] = t;
  }
  rs.item_save.assign(rs.item_rows.size(), -1);
  if (!rs.row_save.empty())
    for (size_t i = 0; i < rs.item_rows.size(); ++i) rs.item_save[i] = rs.row_save[rs.item_rows[i]];
  for (int32_t a = 0; a <= max_adapter; ++a) {
    for (int32_t i = count[a]; i < count[a + 1]; i += kItemRows) {
      rs.item_start.push_back(i);
      rs.item_nrows.push_back(count[a + 1] - i < kItemRows ? count[a + 1] - i : kItemRows);
      rs.item_adapter.push_back(a);
    }
  }
  rs.item_desc.assign(rs.item_start.size() * kItemDescInts, 0);
  for (size_t it = 0; it < rs.item_start.size(); ++it) {
    const int32_t start = rs.item_start[it], nr = rs.item_nrows[it];
    bool contig = true, block_save = nr == kItemRows && rs.item_save[start] >= 0;
    for (int32_t i = 1; i < nr; ++i) {
      if (rs.item_rows[start + i] != rs.item_rows[start] + i) contig = false;
      if (rs.item_save[start + i] != rs.item_save[start] + i) block_save = false;
    }
    int32_t* d = &rs.item_desc[it * kItemDescInts];
    d[0] = start; d[1] = nr; d[2] = rs.item_adapter[it];
    d[3] = (contig ? 1 : 0) | (contig && block_save ? 2 : 0);
    d[4] = rs.item_rows[start]; d[5] = rs.item_save[start];
  }
}

// Validates the table and fills `p`.  Returns MLORA_OK or the error the header documents.
inline mlora_status_t build_plan(const mlora_segment_t* segs, int32_t n_segs, int32_t n_rows,
                                 int32_t n_adapters, HostPlan& p, const int32_t* adapter_rank = nullptr) {
  if (n_segs < 0 || n_rows < 0 || n_adapters < 0 || (n_segs > 0 && segs == nullptr))
    return MLORA_ERR_INVALID_ARG;
  if (adapter_rank)
    for (int32_t a = 0; a < n_adapters; ++a)
      if (adapter_rank[a] < 1 || adapter_rank[a] > kMaxRank) return MLORA_ERR_INVALID_ARG;
  p = HostPlan();
  p.n_rows = n_rows; p.n_adapters = n_adapters; p.n_segs = n_segs;
  if (adapter_rank) p.adapter_rank.assign(adapter_rank, adapter_rank + n_adapters);
  p.fwd.n_rows = n_rows;
  p.fwd.row_adapter.assign(n_rows, -1);
  p.fwd.row_save.assign(n_rows, -1);
  p.seg_save_off.assign(n_segs, -1);
  std::vector<uint8_t> taken(n_rows, 0);
  // pass 1: ranges and adapter ids, so that the error reported does not depend on table order
  for (int32_t k = 0; k < n_segs; ++k) {
    const mlora_segment_t& s = segs[k];
    if (s.row_len < 0 || s.row_start < 0 || (int64_t)s.row_start + s.row_len > n_rows)
      return MLORA_ERR_SEGMENT_RANGE;
    if (s.adapter_id < -1 || s.adapter_id >= n_adapters) return MLORA_ERR_ADAPTER_ID;
    if (s.is_finetune && s.adapter_id < 0) return MLORA_ERR_ADAPTER_ID;
  }
  int32_t off = 0;
  for (int32_t k = 0; k < n_segs; ++k) {
    const mlora_segment_t& s = segs[k];
    for (int32_t i = 0; i < s.row_len; ++i) {
      const int32_t t = s.row_start + i;
      if (taken[t]) return MLORA_ERR_SEGMENT_OVERLAP;
      taken[t] = 1;
      p.fwd.row_adapter[t] = s.adapter_id;
      if (s.is_finetune) p.fwd.row_save[t] = off + i;
    }
    if (s.is_finetune) {
      p.seg_save_off[k] = off;
      off += s.row_len;
      bool seen = false;
      for (int32_t a : p.ft_adapters) seen = seen || (a == s.adapter_id);
      if (!seen) p.ft_adapters.push_back(s.adapter_id);
    }
  }
  p.ft_rows = off;
  build_tiles_and_items(p.fwd);
  if (!p.adapter_rank.empty()) build_ranked(p.fwd, p.adapter_rank);

  // compact fine-tuning row space (save order) and the gradient chunk lists
  p.bwd.n_rows = p.ft_rows;
  p.bwd.row_adapter.assign(p.ft_rows, -1);
  for (int32_t k = 0; k < n_segs; ++k) {
    if (!segs[k].is_finetune) continue;
    for (int32_t i = 0; i < segs[k].row_len; ++i) p.bwd.row_adapter[p.seg_save_off[k] + i] = segs[k].adapter_id;
  }
  build_tiles_and_items(p.bwd);
  if (!p.adapter_rank.empty()) build_ranked(p.bwd, p.adapter_rank);
  p.slot_chunk_off.assign(1, 0);
  for (int32_t a : p.ft_adapters) {
    for (int32_t k = 0; k < n_segs; ++k) {
      if (!segs[k].is_finetune || segs[k].adapter_id != a) continue;
      for (int32_t i = 0; i < segs[k].row_len; i += kChunkRows) {
        p.chunk_row0.push_back(p.seg_save_off[k] + i);
        p.chunk_nrows.push_back(segs[k].row_len - i < kChunkRows ? segs[k].row_len - i : kChunkRows);
      }
    }
    p.slot_chunk_off.push_back((int32_t)p.chunk_row0.size());
  }
  p.slot_blk_off.assign(1, 0);
  for (int32_t a : p.ft_adapters) {
    for (int32_t k = 0; k < n_segs; ++k) {
      if (!segs[k].is_finetune || segs[k].adapter_id != a) continue;
      for (int32_t i = 0; i < segs[k].row_len; i += kTileRows) {
        p.blk_row0.push_back(p.seg_save_off[k] + i);
        p.blk_nrows.push_back(segs[k].row_len - i < kTileRows ? segs[k].row_len - i : kTileRows);
      }
    }
    p.slot_blk_off.push_back((int32_t)p.blk_row0.size());
  }
  if (!p.adapter_rank.empty())
    for (int32_t a : p.ft_adapters) {
      int32_t w = 16;
      while (w < p.adapter_rank[a]) w *= 2;
      p.slot_width.push_back(w);
    }
  return MLORA_OK;
}

}  // namespace mlora
