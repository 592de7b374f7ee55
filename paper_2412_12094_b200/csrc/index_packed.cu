// Index of rows that pack several documents: sepllm_build_index_packed.
//
// Three plain passes (this variant is not on the timed path):
//   packed_scan   one block per row walks it in 8192-token steps, forwards for the document
//                 starts (running maximum of the boundary positions), the side members and their
//                 prefix counts, then backwards for the document ends (running minimum);
//   packed_rows   lim[i] = cnt[max(i-n+1, doc_start[i])] for every position;
//   packed_tiles  one warp per query tile: the eight metadata words; one block writes the header.
#include "attn_common.cuh"

namespace sepllm {

constexpr int kScanThreads = 1024;

// Scan over the block's 1024 values, in thread order or (REVERSE) from the last thread towards the
// first: warp shuffles, then the warps' totals through shared memory (sh: 32 words; two barriers a
// call).  incl includes the thread's own value, excl does not (identity for the first in order).
struct ScanResult {
  int incl, excl;
};
template <bool REVERSE, class Op>
__device__ __forceinline__ ScanResult block_scan(int v, int* sh, Op op, int identity) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  int x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = REVERSE ? __shfl_down_sync(0xffffffffu, x, o) : __shfl_up_sync(0xffffffffu, x, o);
    if (REVERSE ? (lane + o < 32) : (lane >= o)) x = op(x, y);
  }
  if (lane == (REVERSE ? 0 : 31)) sh[w] = x;
  __syncthreads();
  int acc = identity;   // everything in the warps before this one in scan order
  if (REVERSE) { for (int k = kScanThreads / 32 - 1; k > w; --k) acc = op(acc, sh[k]); }
  else { for (int k = 0; k < w; ++k) acc = op(acc, sh[k]); }
  __syncthreads();
  const int nb = REVERSE ? __shfl_down_sync(0xffffffffu, x, 1) : __shfl_up_sync(0xffffffffu, x, 1);
  const bool first_in_warp = REVERSE ? (lane == 31) : (lane == 0);
  ScanResult r;
  r.incl = op(acc, x);
  r.excl = first_in_warp ? acc : op(acc, nb);
  return r;
}

constexpr int kScanItems = 8;                          // consecutive positions per thread
constexpr int kScanStep = kScanThreads * kScanItems;   // positions per step of the walk

__global__ void __launch_bounds__(kScanThreads)
packed_scan(const int32_t* __restrict__ token_ids, const int32_t* __restrict__ doc_first,
            const int32_t* __restrict__ seq_len, SepIds sep, int L, int n_init, int side_cap,
            int32_t* __restrict__ cnt, int32_t* __restrict__ side_pos, int32_t* __restrict__ n_side,
            int32_t* __restrict__ doc_start, int32_t* __restrict__ doc_end,
            int32_t* __restrict__ seq_len_out, int32_t* status) {
  __shared__ int sh[kScanThreads / 32];
  __shared__ int carry_a, carry_b;
  const int b = blockIdx.x, tid = threadIdx.x;
  const int Lv = seq_len ? max(0, min(L, seq_len[b])) : L;
  const int32_t* ids = token_ids + size_t(b) * L;
  const int32_t* df = doc_first + size_t(b) * L;
  int32_t* cnt_b = cnt + size_t(b) * (L + 1);
  int32_t* sp = side_pos + size_t(b) * side_cap;
  int32_t* ds = doc_start + size_t(b) * L;
  int32_t* de = doc_end + size_t(b) * L;
  auto imax = [](int x, int y) { return max(x, y); };
  auto imin = [](int x, int y) { return min(x, y); };
  auto iadd = [](int x, int y) { return x + y; };
  if (tid == 0) { carry_a = 0; carry_b = 0; }   // document start so far, members so far
  __syncthreads();
  // ---- forwards: document starts, members, prefix counts ----
  for (int base = 0; base < L; base += kScanStep) {
    const int j0 = base + tid * kScanItems;
    const int start_before = carry_a, members_before = carry_b;
    // boundaries only grow along the row, so their running maximum is the nearest one so far
    int start[kScanItems], tok[kScanItems];
    int run = -1;
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
      const int j = j0 + k;
      const bool valid = j < Lv;
      tok[k] = valid ? ids[j] : 0;
      if (valid && (j == 0 || df[j] != 0)) run = j;
      start[k] = run;
    }
    const int before = max(block_scan<false>(run, sh, imax, -1).excl, start_before);
    uint32_t member = 0;
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
      const int j = j0 + k;
      const bool valid = j < Lv;
      start[k] = valid ? max(start[k], before) : j;   // padding belongs to no document
      if (valid && (j - start[k] < n_init || is_separator(tok[k], sep))) member |= 1u << k;
    }
    const int n_mine = __popc(member);
    const ScanResult ms = block_scan<false>(n_mine, sh, iadd, 0);
    int c = members_before + ms.excl;
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
      const int j = j0 + k;
      if (j < L) {
        cnt_b[j] = c;
        ds[j] = start[k];
        if ((member >> k) & 1u) {
          if (c < side_cap) sp[c] = j;
          else set_status(status, SEPLLM_CAPACITY_EXCEEDED);
          ++c;
        }
      }
    }
    if (tid == kScanThreads - 1) {   // (every thread read the carries before the scans' barriers)
      carry_a = max(max(run, before), start_before);
      carry_b = members_before + ms.incl;
    }
    __syncthreads();
  }
  const int total = carry_b;
  if (tid == 0) {
    cnt_b[L] = total;
    n_side[b] = total;
    seq_len_out[b] = Lv;
  }
  for (int r = total + tid; r < side_cap; r += kScanThreads) sp[r] = -1;
  // ---- backwards: document ends = the nearest boundary after j, else the end of the row's tokens ----
  __syncthreads();
  if (tid == 0) carry_a = Lv;
  __syncthreads();
  const int n_steps = (L + kScanStep - 1) / kScanStep;
  for (int step = n_steps - 1; step >= 0; --step) {
    const int j0 = step * kScanStep + tid * kScanItems;
    const int end_after = carry_a;
    int nxt[kScanItems];   // nearest boundary after position k among this thread's own positions
    int run = 0x7fffffff;
#pragma unroll
    for (int k = kScanItems - 1; k >= 0; --k) {
      const int j = j0 + k;
      nxt[k] = run;
      if (j < Lv && (j == 0 || df[j] != 0)) run = j;
    }
    const ScanResult sr = block_scan<true>(run, sh, imin, 0x7fffffff);
    const int after = min(sr.excl, end_after);   // boundaries in later threads and later steps
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
      const int j = j0 + k;
      if (j < L) de[j] = (j < Lv) ? min(nxt[k], after) : j;
    }
    __syncthreads();
    if (tid == 0) carry_a = min(sr.incl, end_after);
    __syncthreads();
  }
}

__global__ void __launch_bounds__(256)
packed_rows(const int32_t* __restrict__ cnt, const int32_t* __restrict__ doc_start, int B, int L,
            int n_neighbor, int32_t* __restrict__ lim) {
  const size_t idx = size_t(blockIdx.x) * 256 + threadIdx.x;
  if (idx >= size_t(B) * L) return;
  const int b = int(idx / L), i = int(idx % L);
  const int ws = max(i - n_neighbor + 1, doc_start[idx]);
  lim[idx] = cnt[size_t(b) * (L + 1) + ws];
}

__global__ void __launch_bounds__(128)
packed_tiles(const int32_t* __restrict__ cnt, const int32_t* __restrict__ lim,
             const int32_t* __restrict__ doc_start, const int32_t* __restrict__ seq_len_out, int L,
             int T, int BM, int BN, int n_neighbor, int32_t* __restrict__ tile_meta,
             const __grid_constant__ sepllm_index_header hdr, int32_t* header_out) {
  const int b = blockIdx.y, lane = threadIdx.x & 31;
  const int t = blockIdx.x * 4 + (threadIdx.x >> 5);
  if (blockIdx.x == 0 && blockIdx.y == 0) {
    // header: everything but the status word, which packed_scan may have set
    const int32_t* src = reinterpret_cast<const int32_t*>(&hdr);
    for (int k = 1 + threadIdx.x; k < int(sizeof(hdr) / 4); k += 128) header_out[k] = src[k];
  }
  if (t >= T) return;
  const int Lv = seq_len_out[b];
  int32_t* m = tile_meta + (size_t(b) * T + t) * 8;
  const long long r0 = static_cast<long long>(t) * BM;
  if (r0 >= Lv) {
    if (lane < 8) m[lane] = 0;
    return;
  }
  const int r1 = int(min(static_cast<long long>(Lv), r0 + BM)) - 1;
  const int32_t* cnt_b = cnt + size_t(b) * (L + 1);
  const int32_t* lim_b = lim + size_t(b) * L;
  const int32_t* ds = doc_start + size_t(b) * L;
  int pairs = 0;
  for (int i = int(r0) + lane; i <= r1; i += 32) {
    const int s = ds[i];
    pairs += (lim_b[i] - cnt_b[s]) + (i - max(i - n_neighbor + 1, s) + 1);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) pairs += __shfl_xor_sync(0xffffffffu, pairs, o);
  if (lane == 0) {
    const int s0 = ds[r0];
    const int win_lo = max(int(r0) - n_neighbor + 1, s0), win_hi = r1 + 1;
    m[0] = lim_b[r0] / BN;
    m[1] = (lim_b[r1] + BN - 1) / BN;
    m[2] = win_lo;
    m[3] = win_hi;
    m[4] = win_lo / BN;
    m[5] = (win_hi + BN - 1) / BN;
    m[6] = pairs;
    m[7] = cnt_b[s0] / BN;
  }
}

}  // namespace sepllm

using namespace sepllm;

extern "C" sepllm_status sepllm_build_index_packed(const sepllm_index_desc* desc,
                                                   const int32_t* token_ids,
                                                   const int32_t* doc_first,
                                                   const int32_t* seq_len, const int32_t* sep_ids,
                                                   void* index, void* /*scratch*/, void* stream_) {
  sepllm_index_header h;
  sepllm_status st = fill_index_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (!token_ids || !doc_first || !index || (desc->n_sep > 0 && !sep_ids)) return SEPLLM_INVALID_ARG;
  if (!aligned(index, kAlign) || !aligned(token_ids, 4) || !aligned(doc_first, 4) ||
      (seq_len && !aligned(seq_len, 4)))
    return SEPLLM_INVALID_ARG;
  if (desc->B > 65535) return SEPLLM_UNSUPPORTED;
  h.packed = 1;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  uint8_t* blob = static_cast<uint8_t*>(index);
  SepIds sep;
  sep.n = desc->n_sep;
  for (int k = 0; k < SEPLLM_MAX_SEP_IDS; ++k)
    sep.id[k] = (sep.n > 0) ? sep_ids[(k < sep.n) ? k : 0] : -1;
  auto arr = [&](int64_t off) { return reinterpret_cast<int32_t*>(blob + off); };
  SEPLLM_CUDA_TRY(cudaMemsetAsync(blob, 0, sizeof(sepllm_index_header), stream));
  packed_scan<<<desc->B, kScanThreads, 0, stream>>>(
      token_ids, doc_first, seq_len, sep, desc->L, desc->n_init, desc->side_cap, arr(h.off_cnt),
      arr(h.off_side_pos), arr(h.off_n_side), arr(h.off_doc_start), arr(h.off_doc_end),
      arr(h.off_seq_len), arr(0));
  const size_t n = size_t(desc->B) * desc->L;
  packed_rows<<<unsigned((n + 255) / 256), 256, 0, stream>>>(arr(h.off_cnt), arr(h.off_doc_start),
                                                             desc->B, desc->L, desc->n_neighbor,
                                                             arr(h.off_lim));
  packed_tiles<<<dim3((h.n_tiles + 3) / 4, desc->B), 128, 0, stream>>>(
      arr(h.off_cnt), arr(h.off_lim), arr(h.off_doc_start), arr(h.off_seq_len), desc->L, h.n_tiles,
      desc->BM, desc->BN, desc->n_neighbor, arr(h.off_tile_meta), h, arr(0));
  SEPLLM_CUDA_TRY(cudaGetLastError());
  return SEPLLM_OK;
}
