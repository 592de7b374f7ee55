// Separator index builder: token ids -> cnt / lim / side_pos / n_side / tile_meta.
//
// The mask of Eq. 2 depends on token ids only, so one index serves every head and
// layer.  The token ids are read once:
//   index_scan  : one block per 4096-token chunk.  Flags, block-local prefix counts, and a
//                 decoupled look-back over the earlier chunks' published totals give every
//                 position its global count; the block writes cnt, the shifted copy
//                 lim[i] = cnt[i-n+1], side_pos, and adds its rows' lim values to the kept-pair
//                 count of the query tiles they fall in.  The block that holds a query tile's
//                 first (last) row also writes that tile's metadata, every block fills its share
//                 of the unused end of side_pos, one block writes the header: a single kernel.
// Chunks are handed out by an atomic ticket per sequence, so a block only ever waits on blocks
// that started before it; the wait is bounded all the same.
#include <algorithm>

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

// Membership among the first NS entries of the list (the host pads the list with copies of its
// first id, so NS may exceed the real count).
template <int NS>
__device__ __forceinline__ bool in_sep_list(int32_t tok, const SepIds& s) {
  bool f = false;
#pragma unroll
  for (int k = 0; k < NS; ++k) f |= (tok == s.id[k]);
  return f;
}

// Separator ids as a collision-free multiplicative hash table: slot (id * mult) >> (32 - bits)
// holds the id; empty slots hold the first id (a token equal to it hashes to its own slot, so the
// filler never makes a false match).  One multiply, one shift, one shared-memory load and one
// compare per token instead of one compare per separator id.
constexpr int kSepTableBits = 9;
constexpr int kSepTableSize = 1 << kSepTableBits;
struct SepTable {
  uint32_t mult;
  int32_t slot[kSepTableSize];
};

// Fills `t` for the (non-empty) id list; false if no multiplier of the tried ones separates them.
static bool build_sep_table(const int32_t* ids, int n, SepTable* t) {
  for (uint32_t trial = 0; trial < 4096; ++trial) {
    const uint32_t mult = 0x9E3779B1u * (2 * trial + 1);
    for (int k = 0; k < kSepTableSize; ++k) t->slot[k] = ids[0];
    bool used[kSepTableSize] = {};
    bool ok = true;
    for (int k = 0; k < n && ok; ++k) {
      const uint32_t h = (uint32_t(ids[k]) * mult) >> (32 - kSepTableBits);
      if (used[h] && t->slot[h] != ids[k]) ok = false;  // a repeated id may share its slot
      used[h] = true;
      t->slot[h] = ids[k];
    }
    if (ok) { t->mult = mult; return true; }
  }
  return false;
}

// Scratch words per call: one 64-bit chunk record (state << 32 | count) per chunk, then one
// ticket counter per sequence.  Zeroed before the scan kernel runs.
constexpr uint32_t kChunkAggregate = 1, kChunkPrefix = 2;
inline size_t index_scratch_words(int B, int n_chunks) {
  return 2 * size_t(B) * n_chunks + size_t(B);
}

__device__ __forceinline__ unsigned long long ld_chunk_state(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_chunk_state(unsigned long long* p, uint32_t state, int count) {
  const unsigned long long v = (static_cast<unsigned long long>(state) << 32) | uint32_t(count);
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

constexpr int kLookbackSpins = 1 << 22;
constexpr int kMaxTilesPerChunk = kIdxChunk / kIdxPerThread + 2;  // query tiles of >= 16 rows under one chunk

// Sum of min(i + 1, n) over rows r0..r1.
__device__ __forceinline__ long long window_pairs(int r0, int r1, int n) {
  const long long a = r0 + 1LL, bb = r1 + 1LL;
  const long long k = min(bb, static_cast<long long>(n));
  const long long ramp = (a <= k) ? (a + k) * (k - a + 1) / 2 : 0;
  const long long flat = max(0LL, bb - max(a - 1, static_cast<long long>(n)));
  return ramp + flat * n;
}

// NS >= 0: compare against the first NS list entries; NS == kSepHashed: look the token up in
// `tab`; NS == kByPosition: no token ids, positions that are multiples of `interval` are the
// members (the fixed-interval variant: Section 4.7 and the appendix "Fixed-Interval Variant").
constexpr int kSepHashed = -1, kByPosition = -2;
template <int NS>
__global__ void __launch_bounds__(kIdxThreads, 6)
index_scan(const int32_t* __restrict__ token_ids, int L, int n_init, int n_neighbor, SepIds sep,
           const __grid_constant__ SepTable tab,
           unsigned long long* __restrict__ chunk_state, int32_t* __restrict__ tickets,
           int n_chunks, int side_cap, int32_t* __restrict__ cnt, int32_t* __restrict__ lim,
           int32_t* __restrict__ side_pos, int32_t* __restrict__ n_side,
           int32_t* __restrict__ tile_meta, int T, int BM, int BN, int interval,
           const __grid_constant__ sepllm_index_header hdr, int32_t* status,
           const int32_t* __restrict__ seq_len, int32_t* __restrict__ seq_len_out) {
  __shared__ int warp_buf[kIdxThreads / 32];
  __shared__ int s_chunk, s_off;
  // counts of the chunk, one pad word per 32 so that a thread's 16 consecutive words and a
  // warp's 32 consecutive words are both conflict-free
  __shared__ int32_t cnt_s[kIdxChunk + kIdxChunk / 32];
  __shared__ int32_t tile_part[kMaxTilesPerChunk];
  const int b = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  __shared__ int32_t tab_s[(NS == kSepHashed) ? kSepTableSize : 1];
  __shared__ int lb_sum[kIdxThreads / 32], lb_found[kIdxThreads / 32];
  if (tid == 0) s_chunk = atomicAdd(&tickets[b], 1);
  if (NS == kSepHashed) {
    for (int k = tid; k < kSepTableSize; k += kIdxThreads) tab_s[k] = tab.slot[k];
  }
  __syncthreads();
  auto is_sep = [&](int32_t tok) -> bool {
    if (NS == kSepHashed) return tab_s[(uint32_t(tok) * tab.mult) >> (32 - kSepTableBits)] == tok;
    return in_sep_list<(NS < 0 ? 0 : NS)>(tok, sep);
  };
  const int chunk = s_chunk;
  if (chunk >= n_chunks) return;
  // Rows are divided by BM in several places; BM is a power of two in practice (128 for the
  // attention calls), and a 64-bit division costs about a hundred instructions per thread.
  const bool bm_pow2 = (BM & (BM - 1)) == 0;
  const int bm_log2 = 31 - __clz(BM);
  auto div_bm = [&](long long x) -> long long { return bm_pow2 ? (x >> bm_log2) : x / BM; };
  auto mod_bm = [&](long long x) -> int { return bm_pow2 ? int(x & (BM - 1)) : int(x % BM); };
  const int32_t* ids = token_ids + static_cast<size_t>(b) * L;
  const int base = chunk * kIdxChunk;
  // tokens in this sequence: positions from Lv on are padding (no members, no query rows)
  const int Lv = seq_len ? max(0, min(L, seq_len[b])) : L;

  // flags of this thread's 16 consecutive positions
  const int p0 = tid * kIdxPerThread, j0 = base + p0;
  uint32_t fl = 0;
  if (NS == kByPosition) {
    for (int k = (interval - j0 % interval) % interval; k < kIdxPerThread; k += interval)
      if (j0 + k < L) fl |= 1u << k;
  } else if (j0 + kIdxPerThread <= L && (reinterpret_cast<uintptr_t>(ids + j0) & 15) == 0) {
    const int4* src = reinterpret_cast<const int4*>(ids + j0);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int4 v = src[q];
      fl |= uint32_t(is_sep(v.x)) << (4 * q);
      fl |= uint32_t(is_sep(v.y)) << (4 * q + 1);
      fl |= uint32_t(is_sep(v.z)) << (4 * q + 2);
      fl |= uint32_t(is_sep(v.w)) << (4 * q + 3);
    }
  } else {
#pragma unroll
    for (int k = 0; k < kIdxPerThread; ++k)
      if (j0 + k < L) fl |= uint32_t(is_sep(ids[j0 + k])) << k;
  }
  if (j0 < n_init) {  // initial tokens are side members too
    const int m = max(0, min(kIdxPerThread, min(n_init, L) - j0));
    fl |= (1u << m) - 1u;
  }
  if (j0 + kIdxPerThread > Lv) fl &= (j0 >= Lv) ? 0u : ((1u << (Lv - j0)) - 1u);   // padding holds no members
  const int local = __popc(fl);

  // exclusive scan of `local` over the block
  int incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_buf[wid] = incl;
  __syncthreads();
  int warp_off = 0, total = 0;
#pragma unroll
  for (int k = 0; k < kIdxThreads / 32; ++k) {
    if (k < wid) warp_off += warp_buf[k];
    total += warp_buf[k];
  }

  // publish this chunk's count at once so that later chunks need not wait for its look-back
  unsigned long long* st = chunk_state + static_cast<size_t>(b) * n_chunks;
  if (tid == 0 && chunk > 0) st_chunk_state(st + chunk, kChunkAggregate, total);
  // Position p of the chunk is the lim of row base + shift + p; with BM >= 16 a thread's 16 rows
  // lie in at most two query tiles, whose side-pair sums are gathered in shared memory.
  const int shift = n_neighbor - 1;
  const long long row_lo = static_cast<long long>(base) + shift;
  // (valid rows only: rows of padding count no pairs and belong to no tile with work)
  const int n_rows = int(max(0LL, min(static_cast<long long>(Lv) - row_lo,
                                      static_cast<long long>(min(kIdxChunk, L - base)))));
  const int t_first = int(div_bm(row_lo));
  const bool fast_pairs = (BM >= kIdxPerThread) && (kIdxChunk / BM + 2 <= kMaxTilesPerChunk);
  for (int k = tid; k < kMaxTilesPerChunk; k += kIdxThreads) tile_part[k] = 0;
  __syncthreads();
  {
    int rel = warp_off + incl - local;
    const int kb = BM - mod_bm(row_lo + p0);  // rows k >= kb belong to the next tile
    int s0 = 0, s1 = 0;
    // positions p0 .. p0+15 share p >> 5 (p0 is a multiple of 16): one base address, constant offsets
    int32_t* mine = cnt_s + p0 + (p0 >> 5);
    const int kv = n_rows - p0;   // rows k < kv exist
#pragma unroll
    for (int k = 0; k < kIdxPerThread; ++k) {
      mine[k] = rel;
      const int vv = (k < kv) ? rel : 0;
      s0 += (k < kb) ? vv : 0;
      s1 += (k < kb) ? 0 : vv;
      rel += (fl >> k) & 1u;
    }
    if (fast_pairs) {
      const int tl = int(div_bm(row_lo + p0)) - t_first;
      if (s0) atomicAdd(&tile_part[tl], s0);
      if (s1) atomicAdd(&tile_part[tl + 1], s1);
    }
  }
  // Side members before this chunk: every thread looks at one earlier chunk (warp w at chunks
  // chunk-1-32w .. chunk-32-32w), so the whole look-back is one round trip to L2 when the records
  // are there; a warp waits only for records not yet published.  The sum runs back to the nearest
  // chunk that already holds a prefix.
  {
    int off_acc = 0;
    bool gave_up = false;
    for (int look = chunk - 1; look >= 0; look -= kIdxThreads) {
      const int c = look - tid;
      unsigned long long v = static_cast<unsigned long long>(kChunkPrefix) << 32;  // before chunk 0
      int spins = 0;
      while (true) {
        if (c >= 0) v = ld_chunk_state(st + c);
        if (!__any_sync(0xffffffffu, uint32_t(v >> 32) == 0)) break;
        if (++spins > kLookbackSpins) { gave_up = true; break; }
        __nanosleep(64);
      }
      const uint32_t prefix_mask = __ballot_sync(0xffffffffu, uint32_t(v >> 32) == kChunkPrefix);
      const int first = prefix_mask ? __ffs(prefix_mask) - 1 : 32;
      const int wsum = warp_sum((lane <= first) ? int(uint32_t(v)) : 0);
      __syncthreads();  // the previous round's results have been read
      if (lane == 0) { lb_sum[wid] = wsum; lb_found[wid] = prefix_mask != 0; }
      __syncthreads();
      bool done = false;
#pragma unroll
      for (int w = 0; w < kIdxThreads / 32; ++w) {
        if (!done) off_acc += lb_sum[w];
        done = done || lb_found[w];
      }
      if (done) break;
    }
    if (gave_up) set_status(status, SEPLLM_TIMEOUT);
    if (tid == 0) {
      st_chunk_state(st + chunk, kChunkPrefix, off_acc + total);
      s_off = off_acc;
    }
  }
  __syncthreads();
  const int off = s_off;

  // positions of this thread's side members
  {
    int32_t* sp = side_pos + static_cast<size_t>(b) * side_cap;
    int run = off + warp_off + incl - local;
    uint32_t rest = fl;
    while (rest) {
      const int k = __ffs(rest) - 1;
      rest &= rest - 1;
      if (run < side_cap) sp[run] = j0 + k;
      else set_status(status, SEPLLM_CAPACITY_EXCEEDED);
      ++run;
    }
  }

  int32_t* cnt_b = cnt + static_cast<size_t>(b) * (L + 1);
  int32_t* lim_b = lim + static_cast<size_t>(b) * L;
  if (base + kIdxChunk + shift <= L && base >= shift) {  // whole chunk inside both arrays
    int32_t* cdst = cnt_b + base + tid;
    int32_t* ldst = lim_b + base + shift + tid;
    // position k * 256 + tid sits at word k * 264 + tid + wid of the padded buffer
    const int32_t* src = cnt_s + tid + wid;
#pragma unroll
    for (int k = 0; k < kIdxPerThread; ++k) {
      const int v = src[k * (kIdxThreads + kIdxThreads / 32)] + off;
      cdst[k * kIdxThreads] = v;
      ldst[k * kIdxThreads] = v;
    }
  } else {
#pragma unroll 4
    for (int k = 0; k < kIdxPerThread; ++k) {
      const int p = k * kIdxThreads + tid;
      const int j = base + p;
      if (j < L) {
        const int v = cnt_s[p + (p >> 5)] + off;
        cnt_b[j] = v;
        // lim[i] = cnt[max(0, i-n+1)]: zero for i < n-1, else cnt shifted by n-1
        if (j < shift) lim_b[j] = 0;
        if (static_cast<long long>(j) + shift < L) lim_b[j + shift] = v;
      }
    }
  }
  // Query tiles under this chunk's rows: side pairs (relative sums plus off per row) into word 6,
  // and the rest of the metadata by whoever holds the tile's first row (words 0, 2-5, the window's
  // share of word 6) or last row (word 1).  tile_meta was zeroed before the launch.
  int32_t* meta_b = tile_meta + static_cast<size_t>(b) * T * 8;
  auto window_words = [&](int t) {
    const int r0 = t * BM, r1 = min(Lv, (t + 1) * BM) - 1;
    const int win_lo = max(0, r0 - n_neighbor + 1), win_hi = r1 + 1;
    int32_t* m = meta_b + static_cast<size_t>(t) * 8;
    m[2] = win_lo;
    m[3] = win_hi;
    m[4] = win_lo / BN;
    m[5] = (win_hi + BN - 1) / BN;
    atomicAdd(&m[6], int(window_pairs(r0, r1, n_neighbor)));
  };
  if (n_rows > 0) {
    const long long row_hi = row_lo + n_rows;  // exclusive
    const int t_last = int(div_bm(row_hi - 1));
    for (int t = t_first + (fast_pairs ? tid : wid); t <= t_last; t += (fast_pairs ? kIdxThreads : kIdxThreads / 32)) {
      const long long r0 = max(row_lo, static_cast<long long>(t) * BM);
      const long long r1 = min(row_hi, (static_cast<long long>(t) + 1) * BM);
      int sum;
      if (fast_pairs) {
        sum = tile_part[t - t_first] + off * int(r1 - r0);
      } else {
        sum = 0;
        for (long long r = r0 + lane; r < r1; r += 32) {
          const int p = int(r - row_lo);
          sum += cnt_s[p + (p >> 5)] + off;
        }
        sum = warp_sum(sum);
      }
      if ((fast_pairs || lane == 0)) {
        if (sum) atomicAdd(&meta_b[size_t(t) * 8 + 6], sum);
        const long long first = static_cast<long long>(t) * BM;
        const long long last = min(static_cast<long long>(Lv), first + BM) - 1;
        if (first >= row_lo) {  // this chunk holds the tile's first row
          const int p = int(first - row_lo);
          meta_b[size_t(t) * 8 + 0] = (cnt_s[p + (p >> 5)] + off) / BN;
          window_words(t);
        }
        if (last < row_hi) {    // ... and / or its last row
          const int p = int(last - row_lo);
          meta_b[size_t(t) * 8 + 1] = (cnt_s[p + (p >> 5)] + off + BN - 1) / BN;
        }
      }
    }
  }
  if (chunk == 0) {
    // tiles whose first row comes before row n_neighbor-1 belong to no chunk (lim is 0 there)
    const int Tv = int(div_bm(static_cast<long long>(Lv) + BM - 1));   // tiles that hold tokens
    const int t_head = int(min(static_cast<long long>(Tv), div_bm(static_cast<long long>(shift) + BM - 1)));
    for (int t = tid; t < t_head; t += kIdxThreads) window_words(t);
    if (tid == 0) seq_len_out[b] = Lv;
    if (b == 0) {
      // header: everything but the status word, which any block may be setting
      const int32_t* src = reinterpret_cast<const int32_t*>(&hdr);
      int32_t* dst = status;
      for (int k = 1 + tid; k < int(sizeof(hdr) / 4); k += kIdxThreads) dst[k] = src[k];
    }
  }
  // side_pos beyond n_side reads -1.  If every token after this chunk were a side member the list
  // would end at `bound`; the previous chunk's bound is higher by this chunk's non-members, and
  // that stretch is this block's to fill (chunk 0 fills from its bound to the end of the list).
  {
    const long long end = min(static_cast<long long>(L), static_cast<long long>(base) + kIdxChunk);
    const long long bound = off + total + (L - end);
    const long long upper = (chunk == 0) ? side_cap : min(static_cast<long long>(side_cap),
                                                          static_cast<long long>(off) + (L - base));
    int32_t* sp = side_pos + static_cast<size_t>(b) * side_cap;
    for (long long r = bound + tid; r < upper; r += kIdxThreads) sp[r] = -1;
  }
  if (chunk == n_chunks - 1 && tid == 0) {
    cnt_b[L] = off + total;
    n_side[b] = off + total;
  }
}


// Clears what the scan expects to find zero -- the header (its status word), the chunk records and
// tickets, the tile metadata -- in one launch instead of three memset nodes.
__global__ void __launch_bounds__(256)
index_clear(uint4* __restrict__ header, uint4* __restrict__ tile_meta, size_t meta_words16,
            int32_t* __restrict__ scratch, size_t scratch_words) {
  const size_t i0 = size_t(blockIdx.x) * 256 + threadIdx.x, stride = size_t(gridDim.x) * 256;
  const uint4 z = make_uint4(0, 0, 0, 0);
  if (i0 < sizeof(sepllm_index_header) / 16) header[i0] = z;
  for (size_t i = i0; i < meta_words16; i += stride) tile_meta[i] = z;
  for (size_t i = i0; i < scratch_words; i += stride) scratch[i] = 0;
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
  h->off_seq_len = off;
  off = align_up(off + sizeof(int32_t) * size_t(d->B));
  h->off_doc_start = off;
  off = align_up(off + sizeof(int32_t) * size_t(d->B) * d->L);
  h->off_doc_end = off;
  off = align_up(off + sizeof(int32_t) * size_t(d->B) * d->L);
  h->total_bytes = off;
  return SEPLLM_OK;
}

}  // namespace sepllm

using namespace sepllm;

static_assert(sizeof(sepllm_index_header) == 256, "index header is 256 bytes");

// Launches shared by the two entry points.  `scratch` holds index_scratch_words() int32 words.
static sepllm_status launch_index(const sepllm_index_desc* desc, const sepllm_index_header& h,
                                  const int32_t* token_ids, const int32_t* sep_ids, uint8_t* blob,
                                  int32_t* scratch, cudaStream_t stream, int interval = 0,
                                  const int32_t* seq_len = nullptr) {
  SepIds sep;
  sep.n = desc->n_sep;
  for (int k = 0; k < SEPLLM_MAX_SEP_IDS; ++k)
    sep.id[k] = (sep.n > 0) ? sep_ids[(k < sep.n) ? k : 0] : -1;
  const int n_chunks = (desc->L + kIdxChunk - 1) / kIdxChunk;
  const size_t words = index_scratch_words(desc->B, n_chunks);
  {
    const size_t meta16 = size_t(desc->B) * h.n_tiles * 2;   // eight int32 per tile = two 16-byte words
    const size_t most = std::max(meta16, words);
    const unsigned blocks = unsigned(std::min<size_t>(8 * 148, (most + 255) / 256));
    index_clear<<<std::max(1u, blocks), 256, 0, stream>>>(
        reinterpret_cast<uint4*>(blob), reinterpret_cast<uint4*>(blob + h.off_tile_meta), meta16, scratch,
        words);
  }
  unsigned long long* chunk_state = reinterpret_cast<unsigned long long*>(scratch);
  int32_t* tickets = scratch + 2 * size_t(desc->B) * n_chunks;
  dim3 grid(n_chunks, desc->B);
#define SEPLLM_SCAN(NS)                                                                          \
  index_scan<NS><<<grid, kIdxThreads, 0, stream>>>(                                              \
      token_ids, desc->L, desc->n_init, desc->n_neighbor, sep, tab, chunk_state, tickets,        \
      n_chunks,                                                                                  \
      desc->side_cap, reinterpret_cast<int32_t*>(blob + h.off_cnt),                              \
      reinterpret_cast<int32_t*>(blob + h.off_lim),                                              \
      reinterpret_cast<int32_t*>(blob + h.off_side_pos),                                         \
      reinterpret_cast<int32_t*>(blob + h.off_n_side),                                           \
      reinterpret_cast<int32_t*>(blob + h.off_tile_meta), h.n_tiles, desc->BM, desc->BN,         \
      interval, h, reinterpret_cast<int32_t*>(blob), seq_len,                                    \
      reinterpret_cast<int32_t*>(blob + h.off_seq_len))
  SepTable tab;
  tab.mult = 0;
  const bool hashed = sep.n > 0 && build_sep_table(sep_ids, sep.n, &tab);
  if (interval > 0) SEPLLM_SCAN(kByPosition);
  else if (sep.n == 0) SEPLLM_SCAN(0);
  else if (hashed) SEPLLM_SCAN(kSepHashed);
  else if (sep.n <= 8) SEPLLM_SCAN(8);
  else if (sep.n <= 12) SEPLLM_SCAN(12);
  else if (sep.n <= 16) SEPLLM_SCAN(16);
  else if (sep.n <= 32) SEPLLM_SCAN(32);
  else SEPLLM_SCAN(64);
#undef SEPLLM_SCAN
  SEPLLM_CUDA_TRY(cudaGetLastError());
  return SEPLLM_OK;
}

extern "C" sepllm_status sepllm_index_bytes(const sepllm_index_desc* desc, size_t* index_bytes,
                                            size_t* scratch_bytes) {
  sepllm_index_header h;
  sepllm_status st = fill_index_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (index_bytes) *index_bytes = size_t(h.total_bytes);
  const int n_chunks = (desc->L + kIdxChunk - 1) / kIdxChunk;
  if (scratch_bytes) *scratch_bytes = align_up(sizeof(int32_t) * index_scratch_words(desc->B, n_chunks));
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
  return launch_index(desc, h, token_ids, sep_ids, static_cast<uint8_t*>(index),
                      static_cast<int32_t*>(scratch), static_cast<cudaStream_t>(stream_));
}

extern "C" sepllm_status sepllm_build_index_varlen(const sepllm_index_desc* desc,
                                                   const int32_t* token_ids,
                                                   const int32_t* seq_len, const int32_t* sep_ids,
                                                   void* index, void* scratch, void* stream_) {
  sepllm_index_header h;
  sepllm_status st = fill_index_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (!token_ids || !seq_len || !index || !scratch || (desc->n_sep > 0 && !sep_ids))
    return SEPLLM_INVALID_ARG;
  if (!aligned(index, kAlign) || !aligned(scratch, kAlign) || !aligned(token_ids, 4) ||
      !aligned(seq_len, 4))
    return SEPLLM_INVALID_ARG;
  if (desc->B > 65535) return SEPLLM_UNSUPPORTED;
  return launch_index(desc, h, token_ids, sep_ids, static_cast<uint8_t*>(index),
                      static_cast<int32_t*>(scratch), static_cast<cudaStream_t>(stream_), 0, seq_len);
}

extern "C" sepllm_status sepllm_build_index_fixed_interval(const sepllm_index_desc* desc,
                                                           int32_t interval, void* index,
                                                           void* scratch, void* stream_) {
  sepllm_index_header h;
  sepllm_status st = fill_index_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (interval < 1 || desc->n_sep != 0 || !index || !scratch) return SEPLLM_INVALID_ARG;
  if (!aligned(index, kAlign) || !aligned(scratch, kAlign)) return SEPLLM_INVALID_ARG;
  if (desc->B > 65535) return SEPLLM_UNSUPPORTED;
  return launch_index(desc, h, nullptr, nullptr, static_cast<uint8_t*>(index),
                      static_cast<int32_t*>(scratch), static_cast<cudaStream_t>(stream_), interval);
}

// ---------------------------------------------------------------------------
// Index build without caller-provided scratch
// ---------------------------------------------------------------------------
// The scan's chunk records and tickets for sepllm_build_index_static live in this fixed array
// instead of a caller buffer: 65536 words = 256 KB, held by every device that loads the library
// until exit.  A call needs 2 words per 4096-token chunk plus one per sequence.
constexpr int kStaticWords = 65536;
static __device__ __align__(256) int32_t g_static_chunk_sums[kStaticWords];

// Device address of the array on the current device.  In host code the array's name is only a
// handle, not an address a kernel could use, so the address is looked up on every call (a
// host-side table lookup that allocates nothing): nothing is cached that a re-created context
// could leave dangling.
static sepllm_status static_chunk_sums(int32_t** out) {
  void* p = nullptr;
  SEPLLM_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_chunk_sums));
  if (!p) return SEPLLM_CUDA_ERROR;
  *out = static_cast<int32_t*>(p);
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
  if (index_scratch_words(desc->B, n_chunks) > size_t(kStaticWords)) return SEPLLM_BUFFER_TOO_SMALL;
  int32_t* scratch = nullptr;
  if ((st = static_chunk_sums(&scratch)) != SEPLLM_OK) return st;
  // launch_index clears the words this call uses before the scan reads them, so nothing an
  // earlier call left in the array matters.
  return launch_index(desc, h, token_ids, sep_ids, static_cast<uint8_t*>(index), scratch,
                      static_cast<cudaStream_t>(stream_));
}
