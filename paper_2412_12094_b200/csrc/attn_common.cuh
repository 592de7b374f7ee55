// Declarations shared by the attention translation units.
#pragma once
#include "common.cuh"

namespace sepllm {

constexpr int kBM = 128, kBN = 128;
constexpr uint32_t kTileBlockBytes = 128 * 128;  // 128 rows x 64 bf16, one swizzled block

// Document bounds of an index built for rows that pack several documents
// (sepllm_build_index_packed); all null for any other index.  With them, row i keeps the side
// entries [cnt[doc_start[i]], lim[i]) and the keys from max(i - n + 1, doc_start[i]) to i, and key
// j is kept by queries before doc_end[j] only.
struct DocView {
  const int32_t* cnt;        // [B][L+1]
  const int32_t* doc_start;  // [B][L]
  const int32_t* doc_end;    // [B][L]
};
__device__ __forceinline__ DocView doc_view(const sepllm_index_header* hdr, const int32_t* cnt,
                                            const int32_t* doc_start, const int32_t* doc_end) {
  DocView v;
  const bool packed = hdr->packed != 0;
  v.cnt = packed ? cnt : nullptr;
  v.doc_start = packed ? doc_start : nullptr;
  v.doc_end = packed ? doc_end : nullptr;
  return v;
}

// One query tile of a two-slot CTA (forward and dQ kernels): tile index (-1 = empty slot), query
// head, and the tile's key ranges from tile_meta: side tiles [s0, ns) of which those in
// [full_lo, side_full) are kept in full by every row, window tiles [wlo, whi); ws_last is the
// first window key of the tile's last row.
struct SlotGeom {
  int t, hq, side_full, ns, wlo, whi, s0, full_lo, ws_last;
};
// A tile that starts at or behind the end of its sequence (seq_len from the index) is empty too.
__device__ __forceinline__ SlotGeom load_slot(const int32_t* tile_meta, const int32_t* seq_len, int b,
                                              int T, int t, int hq, int side_tiles_cap,
                                              const DocView& dv, int L, int n_neighbor) {
  SlotGeom g;
  const int len = seq_len[b];
  g.t = (t >= 0 && t * kBM < len) ? t : -1;
  g.hq = hq;
  if (g.t >= 0) {
    const int32_t* meta = tile_meta + (size_t(b) * T + t) * 8;
    g.side_full = meta[0];
    g.ns = min(meta[1], side_tiles_cap);
    g.wlo = meta[4];
    g.whi = meta[5];
    g.s0 = 0;
    g.full_lo = 0;
    g.ws_last = t * kBM + kBM - n_neighbor;
    if (dv.doc_start) {
      const int r1 = min(len, (t + 1) * kBM) - 1;
      const int s = dv.doc_start[size_t(b) * L + r1];
      g.s0 = min(meta[7], g.ns);
      g.full_lo = (dv.cnt[size_t(b) * (L + 1) + s] + kBN - 1) / kBN;
      g.ws_last = max(r1 - n_neighbor + 1, s);
    }
  } else {
    g.side_full = 0; g.ns = 0; g.wlo = 0x3fffffff; g.whi = 0;
    g.s0 = 0x3fffffff; g.full_lo = 0; g.ws_last = 0;
  }
  return g;
}
// Key tile j of the CTA's list (side tiles sbase .. sbase + nsl - 1, then window tiles from wlo)
// is kept by slot g.
__device__ __forceinline__ bool slot_active(const SlotGeom& g, int sbase, int nsl, int wlo, int j) {
  if (j < nsl) return sbase + j >= g.s0 && sbase + j < g.ns;
  const int w = wlo + (j - nsl);
  return w >= g.wlo && w < g.whi;
}

// What one query row keeps: side entries [lo, lim), window keys [ws, row].
struct RowGeom {
  int lim, lo, ws;
};
__device__ __forceinline__ RowGeom row_geom(const int32_t* lim, const DocView& dv, int b, int L,
                                            int row, int n_neighbor, int side_cap) {
  RowGeom r;
  r.lim = 0;
  r.lo = 0;
  r.ws = row - n_neighbor + 1;
  if (row < L) {
    r.lim = min(lim[size_t(b) * L + row], side_cap);
    if (dv.doc_start) {
      const int s = dv.doc_start[size_t(b) * L + row];
      r.lo = min(dv.cnt[size_t(b) * (L + 1) + s], side_cap);
      r.ws = max(r.ws, s);
    }
  }
  return r;
}
// Kept columns [c_lo, c_hi) of one key tile for one row, and whether any row of the query tile
// needs the mask at all.  tile: side tile index, or window tile index (keys tile*kBN ...).
__device__ __forceinline__ void key_range(bool side, int tile, const SlotGeom& g, int row,
                                          const RowGeom& rg, int& c_lo, int& c_hi, bool& need_mask) {
  const int k0 = tile * kBN;
  if (side) {
    c_lo = rg.lo - k0;
    c_hi = rg.lim - k0;
    need_mask = (tile >= g.side_full) || (tile < g.full_lo);
  } else {
    c_lo = rg.ws - k0;
    c_hi = row - k0 + 1;
    need_mask = (k0 + kBN - 1 > g.t * kBM) || (k0 < g.ws_last);
  }
}

struct FwdParams {
  const sepllm_index_header* index_header;   // on the device (its `packed` word is read there)
  const int32_t* cnt;        // [B][L+1]
  const int32_t* lim;        // [B][L]
  const int32_t* tile_meta;  // [B][T][8]
  const int32_t* seq_len;    // [B]
  const int32_t* doc_start;  // [B][L]   (packed index only)
  const int32_t* doc_end;    // [B][L]
  __nv_bfloat16* O;
  float* LSE;
  int32_t* status;
  int L, T, Hq, Hkv, n_neighbor, side_cap, side_tiles_cap, pair_heads;
  int d;                     // row length of Q, K, V and O in memory (<= the kernel's D)
  float scale_log2;
};

// Head sizes between the kernel widths run in the next wider kernel: the tensor maps of Q, K, V and
// dO describe rows of d elements, so the columns from d up to the kernel's D arrive as zeros (they
// add nothing to Q K^T, and give zero columns of O, dQ, dK, dV that are never stored); the side
// buffers and the side-gradient partials have rows of D elements.
inline int kernel_head_dim(int d) { return d <= 64 ? 64 : 128; }

struct AttnLayout {
  int cap_pad;  // side_cap rounded up to 128 rows
  // forward workspace: status | Kside | Vside
  size_t off_ks, off_vs, fwd_bytes;
  // backward workspace: status | Kside | Vside | row statistics (LSE in log2 units, Delta) |
  // dKside | dVside, the last two fp32 [split][B][Hkv][cap_pad][D], D = kernel_head_dim(d)
  size_t off_delta, off_dks, off_dvs, bwd_bytes;
  int split;
};

sepllm_status check_attn(const sepllm_attn_desc* d, const sepllm_index_desc* id);
AttnLayout attn_layout(const sepllm_attn_desc* d, const sepllm_index_desc* id);
sepllm_status fill_index_header(const sepllm_index_desc* d, sepllm_index_header* h);

template <int D>
__global__ void gather_side_kv(const __nv_bfloat16* __restrict__ K,
                               const __nv_bfloat16* __restrict__ V,
                               const int32_t* __restrict__ side_pos,
                               const int32_t* __restrict__ n_side, int L, int d, int Hkv,
                               int side_cap, int cap_pad, __nv_bfloat16* __restrict__ Ks,
                               __nv_bfloat16* __restrict__ Vs, int32_t* __restrict__ status);

// Forward for groups of four query heads at head size 128: two CTAs of a cluster work on the four
// heads of one query tile as one MMA pair (attn_fwd_pair.cu).  Ks64 / K64: maps with 64-row boxes.
sepllm_status launch_fwd_pair(const sepllm_attn_desc* d, const FwdParams& p, int n_tiles,
                              const CUtensorMap& mq, const CUtensorMap& mk64, const CUtensorMap& mv,
                              const CUtensorMap& mks64, const CUtensorMap& mvs, cudaStream_t stream);

// Number of SMs of the current device (persistent kernels launch one CTA per SM).
inline int sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
    return 148;
  return n;
}

// Records desc->events[i] on the stream if the caller asked for it.
inline void record_event(const sepllm_attn_desc* d, int i, cudaStream_t stream) {
  if (d->events && i < d->n_events && d->events[i])
    cudaEventRecord(static_cast<cudaEvent_t>(d->events[i]), stream);
}

// Launches the gather of K/V rows at the side positions into Ks / Vs ([B][Hkv][cap_pad][D]).
// The gather is the first launch of a call that runs it, and it resets the workspace's status word
// (one thread) instead of a memset node in front of it.
void launch_gather(const sepllm_attn_desc* d, const sepllm_index_desc* id, int cap_pad,
                   const void* K, const void* V, const int32_t* side_pos, const int32_t* n_side,
                   void* Ks, void* Vs, int32_t* status, cudaStream_t stream);

}  // namespace sepllm
