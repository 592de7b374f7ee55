// Declarations shared by the attention translation units.
#pragma once
#include "common.cuh"

namespace sepllm {

constexpr int kBM = 128, kBN = 128;
constexpr uint32_t kTileBlockBytes = 128 * 128;  // 128 rows x 64 bf16, one swizzled block

// One query tile of a two-slot CTA (forward and dQ kernels): tile index (-1 = empty slot), query
// head, and the tile's key ranges from tile_meta.
struct SlotGeom {
  int t, hq, side_full, ns, wlo, whi;
};
// A tile that starts at or behind the end of its sequence (seq_len from the index) is empty too.
__device__ __forceinline__ SlotGeom load_slot(const int32_t* tile_meta, const int32_t* seq_len, int b,
                                              int T, int t, int hq, int side_tiles_cap) {
  SlotGeom g;
  g.t = (t >= 0 && t * kBM < seq_len[b]) ? t : -1;
  g.hq = hq;
  if (g.t >= 0) {
    const int32_t* meta = tile_meta + (size_t(b) * T + t) * 8;
    g.side_full = meta[0];
    g.ns = min(meta[1], side_tiles_cap);
    g.wlo = meta[4];
    g.whi = meta[5];
  } else {
    g.side_full = 0; g.ns = 0; g.wlo = 0x3fffffff; g.whi = 0;
  }
  return g;
}
// Key tile j of the CTA's list (side tiles [0, ns), then window tiles from wlo) is kept by slot g.
__device__ __forceinline__ bool slot_active(const SlotGeom& g, int ns, int wlo, int j) {
  if (j < ns) return j < g.ns;
  const int w = wlo + (j - ns);
  return w >= g.wlo && w < g.whi;
}

struct FwdParams {
  const int32_t* lim;        // [B][L]
  const int32_t* tile_meta;  // [B][T][8]
  const int32_t* seq_len;    // [B]
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
                               __nv_bfloat16* __restrict__ Vs);

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
void launch_gather(const sepllm_attn_desc* d, const sepllm_index_desc* id, int cap_pad,
                   const void* K, const void* V, const int32_t* side_pos, const int32_t* n_side,
                   void* Ks, void* Vs, cudaStream_t stream);

}  // namespace sepllm
