// Separator index builder: token ids -> cnt / lim / side_pos / n_side / tile_meta.
//
// The mask of Eq. 2 depends on token ids only, so one index serves every head and
// layer.  Three launches, none of which waits on another block:
//   1. index_count : side-member count of every 4096-token chunk
//   2. index_scan  : chunk offset (sum of earlier chunk counts) + in-chunk prefix scan;
//                    writes cnt, the shifted copy lim[i] = cnt[i-n+1], and side_pos
//   3. index_tiles : per query tile metadata, side_pos tail fill, header
#include <mutex>

#include "common.cuh"

namespace sepllm {

constexpr int kIdxThreads = 256;
constexpr int kIdxPerThread = 16;
constexpr int kIdxChunk = kIdxThreads * kIdxPerThread;  // 4096 tokens per block

__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ int block_sum(int v, int* warp_buf) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  v = warp_sum(v);
  if (lane == 0) warp_buf[wid] = v;
  __syncthreads();
  int t = (lane < (blockDim.x >> 5)) ? warp_buf[lane] : 0;
  t = warp_sum(t);
  __syncthreads();
  return t;
}

__global__ void __launch_bounds__(kIdxThreads)
index_count(const int32_t* __restrict__ token_ids, int L, int n_init, SepIds sep,
            int32_t* __restrict__ chunk_sums, int n_chunks) {
  __shared__ int warp_buf[32];
  const int b = blockIdx.y, chunk = blockIdx.x;
  const int32_t* ids = token_ids + static_cast<size_t>(b) * L;
  const int base = chunk * kIdxChunk;
  int c = 0;
#pragma unroll 4
  for (int k = 0; k < kIdxPerThread; ++k) {
    const int j = base + k * kIdxThreads + threadIdx.x;
    if (j < L) c += (j < n_init) || is_separator(ids[j], sep);
  }
  c = block_sum(c, warp_buf);
  if (threadIdx.x == 0) chunk_sums[b * n_chunks + chunk] = c;
}

__global__ void __launch_bounds__(kIdxThreads)
index_scan(const int32_t* __restrict__ token_ids, int L, int n_init, int n_neighbor, SepIds sep,
           const int32_t* __restrict__ chunk_sums, int n_chunks, int side_cap,
           int32_t* __restrict__ cnt, int32_t* __restrict__ lim, int32_t* __restrict__ side_pos,
           int32_t* __restrict__ n_side, int32_t* status) {
  __shared__ int warp_buf[32];
  __shared__ uint8_t flag_s[kIdxChunk];
  __shared__ int32_t cnt_s[kIdxChunk];
  const int b = blockIdx.y, chunk = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int32_t* ids = token_ids + static_cast<size_t>(b) * L;
  const int base = chunk * kIdxChunk;

  // side members before this chunk
  int off = 0;
  for (int k = tid; k < chunk; k += kIdxThreads) off += chunk_sums[b * n_chunks + k];
  off = block_sum(off, warp_buf);

  // flags, loaded coalesced
#pragma unroll 4
  for (int k = 0; k < kIdxPerThread; ++k) {
    const int p = k * kIdxThreads + tid;
    const int j = base + p;
    flag_s[p] = (j < L) ? uint8_t((j < n_init) || is_separator(ids[j], sep)) : uint8_t(0);
  }
  __syncthreads();

  // each thread owns 16 consecutive positions
  uint8_t fl[kIdxPerThread];
  *reinterpret_cast<uint4*>(fl) = *reinterpret_cast<const uint4*>(&flag_s[tid * kIdxPerThread]);
  int local = 0;
#pragma unroll
  for (int k = 0; k < kIdxPerThread; ++k) local += fl[k];

  // exclusive scan of `local` over the block
  int incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_buf[wid] = incl;
  __syncthreads();
  int warp_off = 0;
  for (int k = 0; k < wid; ++k) warp_off += warp_buf[k];
  int run = off + warp_off + incl - local;

  int32_t* sp = side_pos + static_cast<size_t>(b) * side_cap;
#pragma unroll
  for (int k = 0; k < kIdxPerThread; ++k) {
    const int p = tid * kIdxPerThread + k;
    cnt_s[p] = run;
    if (fl[k]) {
      if (run < side_cap) sp[run] = base + p;
      else set_status(status, SEPLLM_CAPACITY_EXCEEDED);
      ++run;
    }
  }
  __syncthreads();

  int32_t* cnt_b = cnt + static_cast<size_t>(b) * (L + 1);
  int32_t* lim_b = lim + static_cast<size_t>(b) * L;
  const int shift = n_neighbor - 1;
#pragma unroll 4
  for (int k = 0; k < kIdxPerThread; ++k) {
    const int p = k * kIdxThreads + tid;
    const int j = base + p;
    if (j < L) {
      const int v = cnt_s[p];
      cnt_b[j] = v;
      // lim[i] = cnt[max(0, i-n+1)]: zero for i < n-1, else cnt shifted by n-1
      if (j < shift) lim_b[j] = 0;
      if (static_cast<long long>(j) + shift < L) lim_b[j + shift] = v;
    }
  }
  if (chunk == n_chunks - 1 && tid == kIdxThreads - 1) {
    cnt_b[L] = run;  // the last thread's running count is the total
    n_side[b] = run;
  }
}

__global__ void __launch_bounds__(256)
index_tiles(sepllm_index_header hdr, uint8_t* __restrict__ index) {
  const int B = hdr.desc.B, L = hdr.desc.L, n = hdr.desc.n_neighbor;
  const int BM = hdr.desc.BM, BN = hdr.desc.BN, T = hdr.n_tiles, side_cap = hdr.desc.side_cap;
  const int32_t* lim = reinterpret_cast<const int32_t*>(index + hdr.off_lim);
  const int32_t* n_side = reinterpret_cast<const int32_t*>(index + hdr.off_n_side);
  int32_t* side_pos = reinterpret_cast<int32_t*>(index + hdr.off_side_pos);
  int32_t* tile_meta = reinterpret_cast<int32_t*>(index + hdr.off_tile_meta);
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  const int gw = blockIdx.x * warps_per_block + (threadIdx.x >> 5);
  const int n_warps = gridDim.x * warps_per_block;

  if (blockIdx.x == 0 && threadIdx.x == 0) {
    // everything but the status word, which the scan kernel may have set
    sepllm_index_header* out = reinterpret_cast<sepllm_index_header*>(index);
    const int32_t st = out->status;
    *out = hdr;
    out->status = st;
  }

  for (int u = gw; u < B * T; u += n_warps) {
    const int b = u / T, t = u % T;
    const int32_t* lim_b = lim + static_cast<size_t>(b) * L;
    const int r0 = t * BM;
    const int r1 = min(L, (t + 1) * BM) - 1;
    int pairs = 0;
    for (int i = r0 + lane; i <= r1; i += 32) pairs += lim_b[i] + min(i + 1, n);
    pairs = warp_sum(pairs);
    if (lane == 0) {
      int32_t* m = tile_meta + (static_cast<size_t>(b) * T + t) * 8;
      const int win_lo = max(0, r0 - n + 1), win_hi = r1 + 1;
      m[0] = lim_b[r0] / BN;
      m[1] = (lim_b[r1] + BN - 1) / BN;
      m[2] = win_lo;
      m[3] = win_hi;
      m[4] = win_lo / BN;
      m[5] = (win_hi + BN - 1) / BN;
      m[6] = pairs;
      m[7] = 0;
    }
  }

  // side_pos beyond n_side reads -1
  const int gt = blockIdx.x * blockDim.x + threadIdx.x;
  const int n_threads = gridDim.x * blockDim.x;
  for (int b = 0; b < B; ++b) {
    const int ns = min(n_side[b], side_cap);
    for (int r = ns + gt; r < side_cap; r += n_threads)
      side_pos[static_cast<size_t>(b) * side_cap + r] = -1;
  }
}

static sepllm_status check_index_desc(const sepllm_index_desc* d) {
  if (!d) return SEPLLM_INVALID_ARG;
  if (d->B <= 0 || d->L <= 0 || d->n_init < 0 || d->n_neighbor < 1 || d->n_sep < 0 ||
      d->BM <= 0 || d->BN <= 0 || d->side_cap <= 0)
    return SEPLLM_INVALID_ARG;
  if (d->n_sep > SEPLLM_MAX_SEP_IDS) return SEPLLM_UNSUPPORTED;
  return SEPLLM_OK;
}

sepllm_status fill_index_header(const sepllm_index_desc* d, sepllm_index_header* h) {
  sepllm_status st = check_index_desc(d);
  if (st != SEPLLM_OK) return st;
  *h = sepllm_index_header{};
  h->magic = SEPLLM_INDEX_MAGIC;
  h->version = 1;
  h->desc = *d;
  h->n_tiles = (d->L + d->BM - 1) / d->BM;
  size_t off = sizeof(sepllm_index_header);
  h->off_cnt = off;
  off = align_up(off + sizeof(int32_t) * size_t(d->B) * (size_t(d->L) + 1));
  h->off_lim = off;
  off = align_up(off + sizeof(int32_t) * size_t(d->B) * d->L);
  h->off_side_pos = off;
  off = align_up(off + sizeof(int32_t) * size_t(d->B) * d->side_cap);
  h->off_n_side = off;
  off = align_up(off + sizeof(int32_t) * size_t(d->B));
  h->off_tile_meta = off;
  off = align_up(off + sizeof(int32_t) * size_t(d->B) * h->n_tiles * 8);
  h->total_bytes = off;
  return SEPLLM_OK;
}

}  // namespace sepllm

using namespace sepllm;

static_assert(sizeof(sepllm_index_header) == 256, "index header is 256 bytes");

extern "C" sepllm_status sepllm_index_bytes(const sepllm_index_desc* desc, size_t* index_bytes,
                                            size_t* scratch_bytes) {
  sepllm_index_header h;
  sepllm_status st = fill_index_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (index_bytes) *index_bytes = size_t(h.total_bytes);
  const int n_chunks = (desc->L + kIdxChunk - 1) / kIdxChunk;
  if (scratch_bytes) *scratch_bytes = align_up(sizeof(int32_t) * size_t(desc->B) * n_chunks);
  return SEPLLM_OK;
}

extern "C" sepllm_status sepllm_build_index(const sepllm_index_desc* desc,
                                            const int32_t* token_ids, const int32_t* sep_ids,
                                            void* index, void* scratch, void* stream_) {
  sepllm_index_header h;
  sepllm_status st = fill_index_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (!token_ids || !index || !scratch || (desc->n_sep > 0 && !sep_ids)) return SEPLLM_INVALID_ARG;
  if (!aligned(index, kAlign) || !aligned(scratch, kAlign) || !aligned(token_ids, 4))
    return SEPLLM_INVALID_ARG;
  if (desc->B > 65535) return SEPLLM_UNSUPPORTED;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  SepIds sep;
  sep.n = desc->n_sep;
  for (int k = 0; k < SEPLLM_MAX_SEP_IDS; ++k) sep.id[k] = (k < sep.n) ? sep_ids[k] : -1;

  uint8_t* blob = static_cast<uint8_t*>(index);
  const int n_chunks = (desc->L + kIdxChunk - 1) / kIdxChunk;
  int32_t* chunk_sums = static_cast<int32_t*>(scratch);
  SEPLLM_CUDA_TRY(cudaMemsetAsync(blob, 0, sizeof(sepllm_index_header), stream));
  dim3 grid(n_chunks, desc->B);
  index_count<<<grid, kIdxThreads, 0, stream>>>(token_ids, desc->L, desc->n_init, sep, chunk_sums,
                                                n_chunks);
  index_scan<<<grid, kIdxThreads, 0, stream>>>(
      token_ids, desc->L, desc->n_init, desc->n_neighbor, sep, chunk_sums, n_chunks,
      desc->side_cap, reinterpret_cast<int32_t*>(blob + h.off_cnt),
      reinterpret_cast<int32_t*>(blob + h.off_lim),
      reinterpret_cast<int32_t*>(blob + h.off_side_pos),
      reinterpret_cast<int32_t*>(blob + h.off_n_side), reinterpret_cast<int32_t*>(blob));
  const int units = desc->B * h.n_tiles;
  const int blocks = max(1, min(148 * 4, (units + 7) / 8));
  index_tiles<<<blocks, 256, 0, stream>>>(h, blob);
  SEPLLM_CUDA_TRY(cudaGetLastError());
  return SEPLLM_OK;
}

// ---------------------------------------------------------------------------
// Index build without caller-provided scratch
// ---------------------------------------------------------------------------
// Chunk sums for sepllm_build_index_static live in this fixed array instead of a caller buffer.
// 65536 chunks of 4096 ids = 256 KB, held by every device that loads the library until exit.
constexpr int kStaticChunks = 65536;
static __device__ __align__(256) int32_t g_static_chunk_sums[kStaticChunks];

constexpr int kMaxDevices = 64;
static std::mutex g_static_mu;
static int32_t* g_static_ptr[kMaxDevices] = {};

// Device address of the array on the current device.  The array's name is only a host-side
// handle here, so the address is looked up once per device and cached.
static sepllm_status static_chunk_sums(int32_t** out) {
  int dev = -1;
  SEPLLM_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return SEPLLM_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    SEPLLM_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_chunk_sums));
    if (!p) return SEPLLM_CUDA_ERROR;
    g_static_ptr[dev] = static_cast<int32_t*>(p);
  }
  *out = g_static_ptr[dev];
  return SEPLLM_OK;
}

extern "C" sepllm_status sepllm_build_index_static(const sepllm_index_desc* desc,
                                                   const int32_t* token_ids,
                                                   const int32_t* sep_ids, void* index,
                                                   void* stream_) {
  sepllm_index_header h;
  sepllm_status st = fill_index_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (!token_ids || !index || (desc->n_sep > 0 && !sep_ids)) return SEPLLM_INVALID_ARG;
  if (!aligned(index, kAlign) || !aligned(token_ids, 4)) return SEPLLM_INVALID_ARG;
  if (desc->B > 65535) return SEPLLM_UNSUPPORTED;
  const int n_chunks = (desc->L + kIdxChunk - 1) / kIdxChunk;
  if (static_cast<int64_t>(desc->B) * n_chunks > kStaticChunks) return SEPLLM_BUFFER_TOO_SMALL;
  int32_t* chunk_sums = nullptr;
  if ((st = static_chunk_sums(&chunk_sums)) != SEPLLM_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  SepIds sep;
  sep.n = desc->n_sep;
  for (int k = 0; k < SEPLLM_MAX_SEP_IDS; ++k) sep.id[k] = (k < sep.n) ? sep_ids[k] : -1;
  uint8_t* blob = static_cast<uint8_t*>(index);
  SEPLLM_CUDA_TRY(cudaMemsetAsync(blob, 0, sizeof(sepllm_index_header), stream));
  dim3 grid(n_chunks, desc->B);
  // index_count writes every chunk sum that index_scan reads, so nothing left in the array by an
  // earlier call is ever used and nothing has to be cleared.
  index_count<<<grid, kIdxThreads, 0, stream>>>(token_ids, desc->L, desc->n_init, sep, chunk_sums,
                                                n_chunks);
  index_scan<<<grid, kIdxThreads, 0, stream>>>(
      token_ids, desc->L, desc->n_init, desc->n_neighbor, sep, chunk_sums, n_chunks,
      desc->side_cap, reinterpret_cast<int32_t*>(blob + h.off_cnt),
      reinterpret_cast<int32_t*>(blob + h.off_lim),
      reinterpret_cast<int32_t*>(blob + h.off_side_pos),
      reinterpret_cast<int32_t*>(blob + h.off_n_side), reinterpret_cast<int32_t*>(blob));
  const int units = desc->B * h.n_tiles;
  const int blocks = max(1, min(148 * 4, (units + 7) / 8));
  index_tiles<<<blocks, 256, 0, stream>>>(h, blob);
  SEPLLM_CUDA_TRY(cudaGetLastError());
  return SEPLLM_OK;
}
