// Streaming KV cache (Section 3.3): update with compaction, and decode attention.
//
// Physical layout per (sequence, kv head): slots = c + s rows of d bf16.
//   [0, a)        Initial Cache, filled once
//   [a, a+s)      ring: Separator Cache (oldest at sep_start)
//   [a+s, c+s)    ring of c-a rows: neighbour run, oldest at win_start; its newest w entries are
//                 the Local Window Cache, the older ones the Past Window Cache
// Decode walks "virtual" entries 0..Size_run-1 = initial, separator (oldest first), neighbour
// (oldest first) and maps each to its slot, so only retained rows are read.
#include <algorithm>

#include "attn_common.cuh"

namespace sepllm {

struct CacheView {
  sepllm_cache_header* hdr;
  sepllm_cache_seq* seq;
  int64_t* slot_pos;
  uint8_t* slot_is_sep;
};

__host__ __device__ inline CacheView cache_view(void* state, const sepllm_cache_header& h) {
  uint8_t* p = static_cast<uint8_t*>(state);
  CacheView v;
  v.hdr = reinterpret_cast<sepllm_cache_header*>(p);
  v.seq = reinterpret_cast<sepllm_cache_seq*>(p + h.off_seq);
  v.slot_pos = reinterpret_cast<int64_t*>(p + h.off_slot_pos);
  v.slot_is_sep = p + h.off_slot_is_sep;
  return v;
}

static sepllm_status fill_cache_header(const sepllm_cache_desc* d, sepllm_cache_header* h) {
  if (!d) return SEPLLM_INVALID_ARG;
  if (d->B <= 0 || d->Hkv <= 0 || d->Hq <= 0 || d->a < 0 || d->s < 0 || d->w < 1 || d->c < 1)
    return SEPLLM_INVALID_ARG;
  if (!(static_cast<int64_t>(d->a) + d->s + d->w < d->c)) return SEPLLM_INVALID_ARG;
  if (d->Hq % d->Hkv != 0) return SEPLLM_INVALID_ARG;
  if (d->d != 64 && d->d != 128) return SEPLLM_UNSUPPORTED;
  if (d->Hq / d->Hkv > 16) return SEPLLM_UNSUPPORTED;
  if (d->flags & ~SEPLLM_CACHE_FIXED_WINDOW) return SEPLLM_INVALID_ARG;
  *h = sepllm_cache_header{};
  h->magic = SEPLLM_CACHE_MAGIC;
  h->version = 1;
  h->slots = d->c + d->s;
  h->desc = *d;
  size_t off = sizeof(sepllm_cache_header);
  h->off_seq = off;
  off = align_up(off + sizeof(sepllm_cache_seq) * size_t(d->B));
  h->off_slot_pos = off;
  off = align_up(off + sizeof(int64_t) * size_t(d->B) * h->slots);
  h->off_slot_is_sep = off;
  off = align_up(off + size_t(d->B) * h->slots);
  h->total_bytes = off;
  return SEPLLM_OK;
}

// What one update does to a sequence, derived from the state before the update.
struct UpdatePlan {
  int append_slot;   // slot that receives the new token's K/V
  bool compact;      // Size_run reaches c with this token
  int n_past;        // Past Window entries examined by the compaction
  int drop;          // oldest Separator Cache entries (old and moved together) that fall out
};

__device__ __forceinline__ UpdatePlan plan_update(const sepllm_cache_seq& q,
                                                  const sepllm_cache_desc& d) {
  UpdatePlan p;
  p.compact = false;
  p.n_past = 0;
  p.drop = 0;
  if (q.size_init < d.a) {
    p.append_slot = q.size_init;
    return p;
  }
  const int ring = d.c - d.a;
  p.append_slot = d.a + d.s + (q.win_start + q.size_win) % ring;
  const int size_win = q.size_win + 1;
  if (d.flags & SEPLLM_CACHE_FIXED_WINDOW) {
    // fundamental design: the run is the w most recent tokens; what is older leaves at once
    if (size_win > d.w) {
      p.compact = true;
      p.n_past = size_win - d.w;
    }
  } else if (q.size_init + q.size_sep + size_win == d.c) {
    p.compact = true;
    p.n_past = size_win - d.w;
  }
  return p;
}

// Ring starts are below the ring size and v is below the region's entry count, so one conditional
// subtraction wraps the index (no integer division on the decode path).
__device__ __forceinline__ int virtual_to_slot(int v, const sepllm_cache_seq& q,
                                               const sepllm_cache_desc& d) {
  if (v < q.size_init) return v;
  v -= q.size_init;
  if (v < q.size_sep) {
    const int x = q.sep_start + v;
    return d.a + (x >= d.s ? x - d.s : x);
  }
  v -= q.size_sep;
  const int ring = d.c - d.a, x = q.win_start + v;
  return d.a + d.s + (x >= ring ? x - ring : x);
}

constexpr int kUpdThreads = 256;

// Writes the header (passed by value, so nothing on the host has to outlive the launch) and zeroes
// the rest of the state buffer.  grid-stride over 16-byte words; the buffer is 256-byte aligned.
__global__ void __launch_bounds__(256)
cache_init_kernel(sepllm_cache_header h, uint4* __restrict__ state, size_t words16) {
  const uint4* src = reinterpret_cast<const uint4*>(&h);
  constexpr size_t kHdrWords = sizeof(sepllm_cache_header) / 16;
  for (size_t k = size_t(blockIdx.x) * blockDim.x + threadIdx.x; k < words16;
       k += size_t(gridDim.x) * blockDim.x)
    state[k] = (k < kHdrWords) ? src[k] : make_uint4(0, 0, 0, 0);
}

// Exclusive rank of every separator among the Past Window entries, in position order.
// rank_s[k] (k < n_past) = number of separators among past entries [0, k); returns the total.
// n_past <= kMaxPast.
__device__ int rank_past_separators(const uint8_t* slot_is_sep_b, const sepllm_cache_seq& q,
                                    const sepllm_cache_desc& d, int n_past, int16_t* flag_s,
                                    int* warp_buf) {
  const int ring = d.c - d.a;
  const int base = d.a + d.s;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int per = (n_past + kUpdThreads - 1) / kUpdThreads;
  const int k0 = tid * per, k1 = min(n_past, k0 + per);
  int local = 0;
  for (int k = k0; k < k1; ++k) {
    const int f = slot_is_sep_b[base + (q.win_start + k) % ring];
    flag_s[k] = int16_t(f);
    local += f;
  }
  int incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_buf[wid] = incl;
  __syncthreads();
  int woff = 0, total = 0;
  for (int k = 0; k < kUpdThreads / 32; ++k) {
    if (k < wid) woff += warp_buf[k];
    total += warp_buf[k];
  }
  int run = woff + incl - local;
  // flag_s[k] becomes rank+1 for separators, 0 otherwise
  for (int k = k0; k < k1; ++k) {
    if (flag_s[k]) { flag_s[k] = int16_t(run + 1); ++run; }
  }
  __syncthreads();
  return total;
}

constexpr int kMaxPast = 24576;  // int16 ranks in shared memory: 48 KB

// grid (B, Hkv).  Every CTA moves the K/V rows of its kv head (append; at a compaction the ordered
// move of Past-Window separators into the separator ring), reading the sequence's state only.
// The CTA that finishes last for a sequence (an arrival count in the sequence record) then
// updates the per-slot metadata and the record, so the state changes only after every kv head
// has planned its moves from the old one -- one launch instead of two.
//
// ROPE: Kr is a second key buffer with Kc's layout that holds every retained key rotated to its
// current position inside the cache (entry v of the walk initial, separator oldest first,
// neighbour oldest first sits at position v), computed from the un-rotated row in Kc and rounded
// to bf16 once.  An update without a compaction moves nobody, so only the new key is rotated; a
// compaction shifts every entry after the Initial Cache, and the CTA rewrites those rows of its
// kv head from Kc.
template <bool ROPE>
__global__ void __launch_bounds__(kUpdThreads)
cache_update(sepllm_cache_header h, uint8_t* __restrict__ state, __nv_bfloat16* __restrict__ Kc,
             __nv_bfloat16* __restrict__ Vc, const __nv_bfloat16* __restrict__ k_new,
             const __nv_bfloat16* __restrict__ v_new, const int32_t* __restrict__ new_token_ids,
             SepIds sep, __nv_bfloat16* __restrict__ Kr, const float2* __restrict__ rope) {
  extern __shared__ int16_t flag_s[];
  __shared__ int warp_buf[32];
  __shared__ int s_last;
  const sepllm_cache_desc d = h.desc;
  const int b = blockIdx.x, hk = blockIdx.y, tid = threadIdx.x;
  CacheView v = cache_view(state, h);
  const sepllm_cache_seq q = v.seq[b];
  const UpdatePlan p = plan_update(q, d);
  const size_t plane = (size_t(b) * d.Hkv + hk) * h.slots * d.d;
  const int vec = d.d / 8;  // 16-byte chunks per row
  uint4* Kp = reinterpret_cast<uint4*>(Kc + plane);
  uint4* Vp = reinterpret_cast<uint4*>(Vc + plane);
  const uint4* kn = reinterpret_cast<const uint4*>(k_new + (size_t(b) * d.Hkv + hk) * d.d);
  const uint4* vn = reinterpret_cast<const uint4*>(v_new + (size_t(b) * d.Hkv + hk) * d.d);
  if (tid < vec) Kp[size_t(p.append_slot) * vec + tid] = kn[tid];
  else if (tid < 2 * vec) Vp[size_t(p.append_slot) * vec + (tid - vec)] = vn[tid - vec];

  const bool moves = p.compact && d.s > 0;  // the same for every thread of the block
  const int ring = d.c - d.a, wbase = d.a + d.s;
  int m = 0, drop = 0;
  if (moves) {
    m = rank_past_separators(v.slot_is_sep + size_t(b) * h.slots, q, d, p.n_past, flag_s, warp_buf);
    drop = max(0, q.size_sep + m - d.s);
    // `vec` lanes move a K row, the next `vec` lanes the V row
    const int rows_per_pass = kUpdThreads / (2 * vec);
    const int sub = tid / (2 * vec), l = tid % (2 * vec);
    for (int k = sub; k < p.n_past; k += rows_per_pass) {
      const int r = flag_s[k];
      if (r == 0) continue;
      const int fifo = q.size_sep + (r - 1);  // place in the queue of old + moved separators
      if (fifo < drop) continue;              // falls out at once
      const int src = wbase + (q.win_start + k) % ring;
      const int dst = d.a + (q.sep_start + fifo) % d.s;
      if (l < vec) Kp[size_t(dst) * vec + l] = Kp[size_t(src) * vec + l];
      else Vp[size_t(dst) * vec + (l - vec)] = Vp[size_t(src) * vec + (l - vec)];
    }
  }

  // the sequence's record after this update (every CTA derives the same one)
  sepllm_cache_seq nq = q;
  nq.reserved[0] = 0;  // arrival count for the next update
  nq.next_pos = q.next_pos + 1;
  if (q.size_init < d.a) nq.size_init = q.size_init + 1;
  else nq.size_win = q.size_win + 1;
  if (p.compact) {
    if (moves) {
      nq.sep_start = (q.sep_start + drop) % d.s;
      nq.size_sep = q.size_sep + m - drop;
    }
    nq.win_start = (q.win_start + p.n_past) % ring;
    nq.size_win = d.w;
    nq.compactions = q.compactions + 1;
  }

  __syncthreads();  // this CTA's append and moves are visible to all its threads
  if (ROPE) {
    const int size_run = nq.size_init + nq.size_sep + nq.size_win;
    const int v_from = p.compact ? nq.size_init : size_run - 1;
    const int half = vec / 2;  // a thread takes chunk c (elements 8c..8c+7) and its partner c + half
    uint4* Rp = reinterpret_cast<uint4*>(Kr + plane);
    const int items = (size_run - v_from) * half;
    for (int item = tid; item < items; item += kUpdThreads) {
      const int vv = v_from + item / half, c = item % half;
      const int slot = virtual_to_slot(vv, nq, d);
      uint4 lo = Kp[size_t(slot) * vec + c], hi = Kp[size_t(slot) * vec + c + half];
      const float4* cs = reinterpret_cast<const float4*>(rope + size_t(vv) * (d.d / 2) + c * 8);
      __nv_bfloat162* lo2 = reinterpret_cast<__nv_bfloat162*>(&lo);
      __nv_bfloat162* hi2 = reinterpret_cast<__nv_bfloat162*>(&hi);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float4 t4 = cs[e];  // (cos, sin) of pairs 2e and 2e+1
        const float2 x = __bfloat1622float2(lo2[e]), y = __bfloat1622float2(hi2[e]);
        lo2[e] = __floats2bfloat162_rn(x.x * t4.x - y.x * t4.y, x.y * t4.z - y.y * t4.w);
        hi2[e] = __floats2bfloat162_rn(y.x * t4.x + x.x * t4.y, y.y * t4.z + x.y * t4.w);
      }
      Rp[size_t(slot) * vec + c] = lo;
      Rp[size_t(slot) * vec + c + half] = hi;
    }
  }

  // last kv head of the sequence to get here updates the state
  if (tid == 0) {
    __threadfence();
    const int prev = atomicAdd(&v.seq[b].reserved[0], 1);
    s_last = (prev == d.Hkv - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  int64_t* pos_b = v.slot_pos + size_t(b) * h.slots;
  uint8_t* sep_b = v.slot_is_sep + size_t(b) * h.slots;
  if (tid == 0) {
    pos_b[p.append_slot] = q.next_pos;
    sep_b[p.append_slot] = uint8_t(is_separator(new_token_ids[b], sep));
    // a Separator Cache that is not meant to evict did
    if ((d.flags & SEPLLM_CACHE_FIXED_WINDOW) && drop > 0) set_status(&v.hdr->status, SEPLLM_CAPACITY_EXCEEDED);
  }
  if (moves) {
    for (int k = tid; k < p.n_past; k += kUpdThreads) {
      const int r = flag_s[k];
      if (r == 0) continue;
      const int fifo = q.size_sep + (r - 1);
      if (fifo < drop) continue;
      const int src = wbase + (q.win_start + k) % ring;
      const int dst = d.a + (q.sep_start + fifo) % d.s;
      pos_b[dst] = pos_b[src];
      sep_b[dst] = 1;
    }
  }
  if (tid == 0) v.seq[b] = nq;
}

// ---------------------------------------------------------------------------
// Prompt hand-off: the cache a pre-filled prompt leaves for generation
// ---------------------------------------------------------------------------
// Taking a prompt in token by token leaves (i) the first a positions in the Initial Cache, (ii) a
// neighbour run that is the contiguous stretch [lo, T) of positions, and (iii) in the Separator
// Cache the newest (at most s) separators of [a, lo): every compaction appends the separators it
// passes in position order and keeps the newest s, and a tail of a tail is a tail.  Only lo needs
// the history: a compaction happens when a + Size_sep + (t - lo) reaches c, and it moves lo to
// t - w.  The separator counts this needs are differences of the index's prefix count `cnt`.
constexpr int kPlanThreads = 1024;

struct PromptPlan {
  int size_init, size_sep, size_win, lo, compactions;
};

// grid B.  Writes the sequence record and the per-slot position / separator flag of one sequence;
// block 0 also writes the header.  Rings start at 0.
__global__ void __launch_bounds__(kPlanThreads)
prompt_plan(sepllm_cache_header h, uint8_t* __restrict__ state, const uint8_t* __restrict__ index,
            sepllm_index_header ih, const int32_t* __restrict__ prompt_len) {
  __shared__ PromptPlan s_plan;
  __shared__ int s_bad;
  const sepllm_cache_desc d = h.desc;
  const int b = blockIdx.x, tid = threadIdx.x;
  const int L = ih.desc.L;
  CacheView v = cache_view(state, h);
  const int32_t* cnt = reinterpret_cast<const int32_t*>(index + ih.off_cnt) + size_t(b) * (L + 1);
  const int32_t* side_pos =
      reinterpret_cast<const int32_t*>(index + ih.off_side_pos) + size_t(b) * ih.desc.side_cap;
  if (tid == 0) {
    const sepllm_index_header* dev = reinterpret_cast<const sepllm_index_header*>(index);
    bool bad = dev->magic != SEPLLM_INDEX_MAGIC || dev->desc.B != ih.desc.B ||
               dev->desc.L != ih.desc.L || dev->desc.n_init != ih.desc.n_init ||
               dev->desc.side_cap != ih.desc.side_cap ||
               dev->packed != 0;   // an index of packed rows describes no single prompt
    int T = L;
    if (prompt_len) {
      T = prompt_len[b];
      if (T < 0 || T > L) { bad = true; T = max(0, min(T, L)); }
    }
    if (bad) T = 0;
    PromptPlan p;
    p.size_init = min(T, d.a);
    p.size_sep = 0;
    p.lo = d.a;
    p.compactions = 0;
    bool overflow = false;
    if (T > d.a && (d.flags & SEPLLM_CACHE_FIXED_WINDOW)) {
      // fundamental design: the run is the last w tokens, every separator before it is kept
      p.lo = max(d.a, T - d.w);
      const int n_sep = cnt[p.lo] - cnt[d.a];
      p.size_sep = min(d.s, n_sep);
      overflow = d.s > 0 && n_sep > d.s;
      p.compactions = p.lo - d.a;
    } else if (T > d.a) {
      const int period = d.c - d.a - d.s - d.w;
      for (;;) {
        const int64_t t_full = int64_t(d.c) - d.a - p.size_sep + p.lo;  // tokens seen when Size_run = c
        if (t_full > T) break;
        const int nlo = int(t_full) - d.w;
        if (d.s > 0) p.size_sep = min(d.s, p.size_sep + (cnt[nlo] - cnt[p.lo]));
        p.lo = nlo;
        ++p.compactions;
        if (p.size_sep == d.s) {  // full for good: the remaining compactions are `period` apart
          const int k = int((T - t_full) / period);
          p.lo += k * period;
          p.compactions += k;
          break;
        }
      }
    }
    p.size_win = max(0, T - p.lo);
    s_plan = p;
    s_bad = bad;
    sepllm_cache_seq q{};
    q.size_init = p.size_init;
    q.size_sep = p.size_sep;
    q.size_win = p.size_win;
    q.compactions = p.compactions;
    q.next_pos = T;
    v.seq[b] = q;
    if (bad) atomicExch(&v.hdr->status, SEPLLM_INVALID_ARG);
    else if (overflow) set_status(&v.hdr->status, SEPLLM_CAPACITY_EXCEEDED);
  }
  if (b == 0) {
    // header: everything but the status word, which a failing block may be writing
    const int32_t* src = reinterpret_cast<const int32_t*>(&h);
    int32_t* dst = reinterpret_cast<int32_t*>(v.hdr);
    for (int k = 1 + tid; k < int(sizeof(h) / 4); k += kPlanThreads) dst[k] = src[k];
  }
  __syncthreads();
  const PromptPlan p = s_plan;
  int64_t* pos_b = v.slot_pos + size_t(b) * h.slots;
  uint8_t* sep_b = v.slot_is_sep + size_t(b) * h.slots;
  const int first_rank = p.size_sep > 0 ? cnt[p.lo] - p.size_sep : 0;  // among the index's side members
  for (int slot = tid; slot < h.slots; slot += kPlanThreads) {
    int64_t pos = 0;
    int flag = 0;
    if (slot < d.a) {
      if (slot < p.size_init) pos = slot;
    } else if (slot < d.a + d.s) {
      const int k = slot - d.a;
      if (k < p.size_sep) {
        // the side member of rank r: the index's side list has it unless the list was cut short,
        // then it is the smallest j with cnt[j + 1] > r
        const int r = first_rank + k;
        if (r < ih.desc.side_cap) {
          pos = side_pos[r];
        } else {
          int lo = d.a, hi = p.lo - 1;
          while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (cnt[mid + 1] > r) hi = mid; else lo = mid + 1;
          }
          pos = lo;
        }
        flag = 1;
      }
    } else {
      const int k = slot - d.a - d.s;
      if (k < p.size_win) {
        pos = p.lo + k;
        flag = cnt[p.lo + k + 1] - cnt[p.lo + k];
      }
    }
    pos_b[slot] = pos;
    sep_b[slot] = uint8_t(flag);
  }
}

constexpr int kCopyThreads = 256;
constexpr int kCopyRows = 64;  // slots per CTA

// grid (ceil(slots / kCopyRows), Hkv, B).  Copies the K and V rows of the retained positions into
// their slots; 2 * D/8 lanes move one slot's K row and V row in 16-byte pieces.  ROPE: the K lanes
// also write the row rotated to its position inside the cache into Kr (rings start at slot 0, so
// the position follows from the slot).
template <int D, bool ROPE>
__global__ void __launch_bounds__(kCopyThreads)
prompt_copy(sepllm_cache_header h, const uint8_t* __restrict__ state,
            const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V, int L,
            __nv_bfloat16* __restrict__ Kc, __nv_bfloat16* __restrict__ Vc,
            __nv_bfloat16* __restrict__ Kr, const float2* __restrict__ rope) {
  constexpr int kVec = D / 8;
  constexpr int kRowsPerPass = kCopyThreads / (2 * kVec);
  const sepllm_cache_desc d = h.desc;
  const int b = blockIdx.z, hk = blockIdx.y, tid = threadIdx.x;
  CacheView v = cache_view(const_cast<uint8_t*>(state), h);
  const sepllm_cache_seq q = v.seq[b];
  const int64_t* pos_b = v.slot_pos + size_t(b) * h.slots;
  const size_t src_plane = (size_t(b) * d.Hkv + hk) * size_t(L) * kVec;
  const size_t dst_plane = (size_t(b) * d.Hkv + hk) * size_t(h.slots) * kVec;
  const int sub = tid / (2 * kVec), l = tid % (2 * kVec);
  const bool is_v = l >= kVec;
  const int ch = is_v ? l - kVec : l;  // 16-byte chunk of the row
  const uint4* src = reinterpret_cast<const uint4*>(is_v ? V : K) + src_plane;
  uint4* dst = reinterpret_cast<uint4*>(is_v ? Vc : Kc) + dst_plane;
  uint4* rdst = reinterpret_cast<uint4*>(Kr) + dst_plane;
  const int slot0 = blockIdx.x * kCopyRows;
#pragma unroll 4
  for (int r = sub; r < kCopyRows; r += kRowsPerPass) {
    const int slot = slot0 + r;
    if (slot >= h.slots) break;
    const bool used = slot < d.a ? slot < q.size_init
                    : slot < d.a + d.s ? slot - d.a < q.size_sep
                                       : slot - d.a - d.s < q.size_win;
    if (!used) continue;
    const uint4* row = src + size_t(pos_b[slot]) * kVec;
    uint4 mine = __ldg(row + ch);
    dst[size_t(slot) * kVec + ch] = mine;
    if (ROPE && !is_v) {
      // chunk ch holds elements 8ch..8ch+7; its partner in the rotation is the chunk half a row away
      const int vpos = slot < d.a ? slot
                     : slot < d.a + d.s ? q.size_init + (slot - d.a)
                                        : q.size_init + q.size_sep + (slot - d.a - d.s);
      uint4 other = __ldg(row + (ch ^ (kVec / 2)));
      const float4* cs = reinterpret_cast<const float4*>(rope + size_t(vpos) * (D / 2) + (ch % (kVec / 2)) * 8);
      const float sgn = (ch < kVec / 2) ? -1.f : 1.f;  // first half: x cos - y sin; second: x cos + y sin
      __nv_bfloat162* x2 = reinterpret_cast<__nv_bfloat162*>(&mine);
      const __nv_bfloat162* y2 = reinterpret_cast<const __nv_bfloat162*>(&other);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float4 t4 = cs[e];
        const float2 x = __bfloat1622float2(x2[e]), y = __bfloat1622float2(y2[e]);
        x2[e] = __floats2bfloat162_rn(x.x * t4.x + sgn * y.x * t4.y, x.y * t4.z + sgn * y.y * t4.w);
      }
      rdst[size_t(slot) * kVec + ch] = mine;
    }
  }
}

// ---------------------------------------------------------------------------
// Decode: one query per sequence over the retained entries
// ---------------------------------------------------------------------------
constexpr int kDecThreads = 128;

// ---- warp-level MMA pieces used by the decode kernel (bf16 inputs, fp32 accumulation) ----
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0,
                                          uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
      "{%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
// 16-byte asynchronous copy; src_bytes = 0 writes zeros.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

constexpr int kDecStages = 2;
constexpr int kDecTile = 16;  // cache rows per warp tile

template <int D>
constexpr int decode_smem_bytes() {
  // per warp: kDecStages x (K tile + V tile); reused after the loop for the warps' partial results
  return (kDecThreads / 32) * kDecStages * 2 * kDecTile * D * 2;
}

// grid (splits, Hkv, B), 4 warps.  HBM-bound: the kernel exists to stream every retained K/V row
// once.  Each warp is an independent flash-decoding worker over its share of the split's rows:
// 16-row K and V tiles arrive through a 2-stage cp.async ring (64 KB per CTA, three CTAs per SM) (virtual entry -> slot mapping done
// per row; rows past the end are zero-filled), the G query heads of the kv head sit in the M
// dimension of warp-level MMAs (rows G..15 are zero), scores go through an online softmax with a
// lazily moved reference, and O accumulates in registers.  The four warps' partials are merged
// through shared memory into one (m, l, acc) record per (query head, split).
//
// ROPE: Kc is the rotated key buffer that the update keeps (every key already turned to its
// position inside the cache, entry v of the walk above at position v) and q arrives un-rotated:
// it is rotated to position Size_run - 1, pair (i, i + D/2) by the angle (Size_run - 1) * theta_i
// from a table of (cos, sin) per (position, i), while its fragments load.
//
// WIDE: groups of 9 to 16 query heads per kv head use both row halves of the MMA tile (a lane
// then carries the softmax state of rows frow and frow + 8); narrower groups leave the upper
// half zero and skip its arithmetic.
template <int D, bool ROPE, bool WIDE>
__global__ void __launch_bounds__(kDecThreads, 3)   // three CTAs per SM: at most 168 registers
decode_split(sepllm_cache_header h, float scale_log2, const __nv_bfloat16* __restrict__ q_in,
             const uint8_t* __restrict__ state, const __nv_bfloat16* __restrict__ Kc,
             const __nv_bfloat16* __restrict__ Vc, float* __restrict__ part_ml,
             float* __restrict__ part_acc, int splits, const float2* __restrict__ rope,
             int32_t* __restrict__ status) {
  constexpr int CH = D / 8;                 // 16-byte chunks per row
  constexpr int ROWB = D * 2;               // bytes per row
  constexpr int TILEB = kDecTile * ROWB;    // bytes of one K (or V) tile
  constexpr int NW = kDecThreads / 32;
  constexpr int RPP = 32 / CH;              // rows covered by one pass of the warp's copies
  constexpr int RH = WIDE ? 2 : 1;          // row halves of the 16-row MMA tile in use
  constexpr int GS = 8 * RH;                // rows per warp in the merge buffers
  extern __shared__ __align__(128) uint8_t dec_smem[];
  const sepllm_cache_desc d = h.desc;
  const int G = d.Hq / d.Hkv;
  const int split = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  if (tid == 0 && (split | hk | b) == 0) *status = SEPLLM_OK;
  CacheView cv = cache_view(const_cast<uint8_t*>(state), h);
  const sepllm_cache_seq sq = cv.seq[b];
  const int size_run = sq.size_init + sq.size_sep + sq.size_win;
  const int per = ((size_run + splits - 1) / splits + kDecTile - 1) / kDecTile * kDecTile;
  const int v0 = split * per, v1 = min(size_run, v0 + per);
  const int n_tiles = (v1 > v0) ? (v1 - v0 + kDecTile - 1) / kDecTile : 0;
  const int my_n = (n_tiles > wid) ? (n_tiles - wid + NW - 1) / NW : 0;  // tiles wid, wid+NW, ...

  const size_t plane = (size_t(b) * d.Hkv + hk) * h.slots * D;
  const uint8_t* Kp = reinterpret_cast<const uint8_t*>(Kc + plane);
  const uint8_t* Vp = reinterpret_cast<const uint8_t*>(Vc + plane);
  uint8_t* wbase = dec_smem + wid * (kDecStages * 2 * TILEB);
  const uint32_t wbase_u = smem_u32(wbase);

  // Q fragments (A operand, row = query head of the group): registers 0 and 2 of each k-step
  const int frow = lane >> 2, fcol = (lane & 3) * 2;
  uint32_t qa[D / 16][4];
  {
    // two consecutive elements e, e+1 of a (rotated) query row as packed bf16
    const __nv_bfloat16* q_lo = q_in + (size_t(b) * d.Hq + hk * G + min(frow, G - 1)) * D;
    const __nv_bfloat16* q_hi = q_in + (size_t(b) * d.Hq + hk * G + min(frow + 8, G - 1)) * D;
    auto q_pair = [&](const __nv_bfloat16* qrow, int e) -> uint32_t {
      if (!ROPE) return *reinterpret_cast<const uint32_t*>(qrow + e);
      const int i = e % (D / 2);
      const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(qrow + e));
      const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(qrow + (e ^ (D / 2))));
      const float2 cs0 = rope[size_t(size_run - 1) * (D / 2) + i];
      const float2 cs1 = rope[size_t(size_run - 1) * (D / 2) + i + 1];
      const float sgn = (e < D / 2) ? -1.f : 1.f;  // first half: x cos - y sin; second: x cos + y sin
      return pack_bf16(x.x * cs0.x + sgn * y.x * cs0.y, x.y * cs1.x + sgn * y.y * cs1.y);
    };
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      const bool lo = frow < G && size_run > 0, hi = WIDE && frow + 8 < G && size_run > 0;
      qa[ks][0] = lo ? q_pair(q_lo, ks * 16 + fcol) : 0u;
      qa[ks][2] = lo ? q_pair(q_lo, ks * 16 + 8 + fcol) : 0u;
      qa[ks][1] = hi ? q_pair(q_hi, ks * 16 + fcol) : 0u;
      qa[ks][3] = hi ? q_pair(q_hi, ks * 16 + 8 + fcol) : 0u;
    }
  }

  // copies of tile `i` (this warp's i-th) into stage i % kDecStages
  const int crow = lane / CH, cch = lane % CH;
  auto issue = [&](int i) {
    const int tile = wid + i * NW;
    const int vbase = v0 + tile * kDecTile;
    const uint32_t sK = wbase_u + (i % kDecStages) * 2 * TILEB, sV = sK + TILEB;
#pragma unroll
    for (int pss = 0; pss < kDecTile / RPP; ++pss) {
      const int r = pss * RPP + crow;
      const int v = vbase + r;
      const bool valid = v < v1;
      const int slot = virtual_to_slot(valid ? v : v1 - 1, sq, d);
      const uint32_t off = uint32_t(r) * ROWB + (uint32_t(cch ^ (r & 7)) << 4);
      const size_t goff = size_t(slot) * ROWB + cch * 16;
      cp_async16(sK + off, Kp + goff, valid ? 16u : 0u);
      cp_async16(sV + off, Vp + goff, valid ? 16u : 0u);
    }
  };

  float oacc[D / 8][4];
#pragma unroll
  for (int n = 0; n < D / 8; ++n)
#pragma unroll
    for (int e = 0; e < 4; ++e) oacc[n][e] = 0.f;
  // of rows frow (+ 8): reference exponent and this lane's share of the row sum
  float m_ref[RH], l_part[RH];
#pragma unroll
  for (int r = 0; r < RH; ++r) { m_ref[r] = -INFINITY; l_part[r] = 0.f; }

#pragma unroll
  for (int s = 0; s < kDecStages - 1; ++s) {
    if (s < my_n) issue(s);
    cp_async_commit();
  }
  for (int i = 0; i < my_n; ++i) {
    cp_async_wait<kDecStages - 2>();
    __syncwarp();
    if (i + kDecStages - 1 < my_n) issue(i + kDecStages - 1);
    cp_async_commit();

    const uint32_t sK = wbase_u + (i % kDecStages) * 2 * TILEB, sV = sK + TILEB;
    // S[16 heads x 16 rows] = Q K^T
    float sc[2][4];
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) sc[n][e] = 0.f;
    {
      const int key = (lane & 7) + ((lane >> 4) << 3);
      const int chb = (lane >> 3) & 1;
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        uint32_t kb[4];
        ldsm_x4(sK + key * ROWB + (uint32_t((2 * ks + chb) ^ (key & 7)) << 4), kb);
        mma_16816(sc[0], qa[ks], kb[0], kb[1]);
        mma_16816(sc[1], qa[ks], kb[2], kb[3]);
      }
    }
    // online softmax over the 16 cache rows of the tile for query heads frow (and frow + 8)
    const int vbase = v0 + (wid + i * NW) * kDecTile;
    uint32_t pa[4] = {0u, 0u, 0u, 0u};
    float corr[RH];
    bool rescale = false;
#pragma unroll
    for (int r = 0; r < RH; ++r) {
      float sv[4];
#pragma unroll
      for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int v = vbase + n * 8 + fcol + e;
          sv[n * 2 + e] = (v < v1) ? sc[n][2 * r + e] * scale_log2 : -INFINITY;
        }
      float mx = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      corr[r] = 1.f;
      if (mx > m_ref[r] + 8.f) {  // lazy: the reference moves only when the maximum grew by > 2^8
        corr[r] = (m_ref[r] == -INFINITY) ? 0.f : ex2(m_ref[r] - mx);
        m_ref[r] = mx;
        rescale = true;
      }
      const float m_eff = (m_ref[r] == -INFINITY) ? 0.f : m_ref[r];
      const float p0 = ex2(sv[0] - m_eff), p1 = ex2(sv[1] - m_eff);
      const float p2 = ex2(sv[2] - m_eff), p3 = ex2(sv[3] - m_eff);
      l_part[r] = l_part[r] * corr[r] + (p0 + p1) + (p2 + p3);
      pa[r] = pack_bf16(p0, p1);
      pa[2 + r] = pack_bf16(p2, p3);
    }
    if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
      for (int n = 0; n < D / 8; ++n)
#pragma unroll
        for (int r = 0; r < RH; ++r) { oacc[n][2 * r] *= corr[r]; oacc[n][2 * r + 1] *= corr[r]; }
    }
    // O[16 heads x D] += P V
    {
      const int key = (lane & 7) + (((lane >> 3) & 1) << 3);
      const int chb = lane >> 4;
#pragma unroll
      for (int j = 0; j < CH; j += 2) {
        uint32_t vb[4];
        ldsm_x4_trans(sV + key * ROWB + (uint32_t((j + chb) ^ (key & 7)) << 4), vb);
        mma_16816(oacc[j], pa, vb[0], vb[1]);
        mma_16816(oacc[j + 1], pa, vb[2], vb[3]);
      }
    }
    __syncwarp();  // every lane is done with this stage before a later copy overwrites it
  }
  cp_async_wait<0>();
#pragma unroll
  for (int r = 0; r < RH; ++r) {
    l_part[r] += __shfl_xor_sync(0xffffffffu, l_part[r], 1);
    l_part[r] += __shfl_xor_sync(0xffffffffu, l_part[r], 2);
  }
  __syncthreads();  // all warps are out of their stage buffers

  // merge the warps' partials: sm_ml[w][g] = (m, l), sm_acc[w][g][D]
  float2* sm_ml = reinterpret_cast<float2*>(dec_smem);
  float* sm_acc = reinterpret_cast<float*>(dec_smem + NW * GS * sizeof(float2));
#pragma unroll
  for (int r = 0; r < RH; ++r) {
    const int g = frow + 8 * r;
    if (g < G) {
      if ((lane & 3) == 0) sm_ml[wid * GS + g] = make_float2(m_ref[r], l_part[r]);
#pragma unroll
      for (int n = 0; n < D / 8; ++n)
        *reinterpret_cast<float2*>(sm_acc + (wid * GS + g) * D + n * 8 + fcol) =
            make_float2(oacc[n][2 * r], oacc[n][2 * r + 1]);
    }
  }
  __syncthreads();
  for (int idx = tid; idx < G * D; idx += kDecThreads) {
    const int g = idx / D, e = idx % D;
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < NW; ++w) mm = fmaxf(mm, sm_ml[w * GS + g].x);
    float ll = 0.f, aa = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float2 ml = sm_ml[w * GS + g];
      const float scf = (ml.x == -INFINITY) ? 0.f : ex2(ml.x - mm);
      ll += ml.y * scf;
      aa += sm_acc[(w * GS + g) * D + e] * scf;
    }
    const size_t uo = ((size_t(b) * d.Hq + hk * G + g) * splits + split);
    part_acc[uo * D + e] = aa;
    if (e == 0) { part_ml[uo * 2] = mm; part_ml[uo * 2 + 1] = ll; }
  }
}

// grid (Hq, B), D threads.
template <int D>
__global__ void decode_combine(sepllm_cache_header h, const float* __restrict__ part_ml,
                               const float* __restrict__ part_acc, int splits,
                               __nv_bfloat16* __restrict__ o, float* __restrict__ lse) {
  const int hq = blockIdx.x, b = blockIdx.y, e = threadIdx.x;
  const size_t u0 = (size_t(b) * h.desc.Hq + hq) * splits;
  float mm = -INFINITY;
  for (int s = 0; s < splits; ++s) mm = fmaxf(mm, part_ml[(u0 + s) * 2]);
  float ll = 0.f, aa = 0.f;
  for (int s = 0; s < splits; ++s) {
    const float ms = part_ml[(u0 + s) * 2];
    const float sc = (ms == -INFINITY) ? 0.f : ex2(ms - mm);
    ll += part_ml[(u0 + s) * 2 + 1] * sc;
    aa += part_acc[(u0 + s) * D + e] * sc;
  }
  const size_t row = size_t(b) * h.desc.Hq + hq;
  o[row * D + e] = __float2bfloat16(ll > 0.f ? aa / ll : 0.f);
  if (lse && e == 0) lse[row] = (ll > 0.f) ? (mm + log2f(ll)) * 0.6931471805599453f : -INFINITY;
}

// (cos, sin) of position * base^(-2i/D) for every position a cache entry can have and every
// pair index i < D/2.
__global__ void rope_table_kernel(float2* __restrict__ table, int positions, int half_d,
                                  float log2_base) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= positions * half_d) return;
  const int pos = idx / half_d, i = idx % half_d;
  const float theta = exp2f(-log2_base * float(i) / float(half_d));
  float sn, cs;
  sincosf(float(pos) * theta, &sn, &cs);
  table[idx] = make_float2(cs, sn);
}

static int decode_splits(const sepllm_cache_desc* d) {
  // about four CTAs per SM over the whole grid, each with at least 256 rows (64 per warp)
  const int units = d->B * d->Hkv;
  int s = (148 * 4 + units - 1) / units;
  const int max_by_rows = (d->c + 255) / 256;
  if (s > max_by_rows) s = max_by_rows;
  if (s < 1) s = 1;
  if (s > 64) s = 64;
  return s;
}

}  // namespace sepllm

using namespace sepllm;

static_assert(sizeof(sepllm_cache_header) == 256, "cache header is 256 bytes");
static_assert(sizeof(sepllm_cache_seq) == 64, "sequence record is 64 bytes");

extern "C" sepllm_status sepllm_cache_bytes(const sepllm_cache_desc* desc, size_t* state_bytes,
                                            size_t* kv_bytes) {
  sepllm_cache_header h;
  sepllm_status st = fill_cache_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (state_bytes) *state_bytes = size_t(h.total_bytes);
  if (kv_bytes) *kv_bytes = size_t(desc->B) * desc->Hkv * h.slots * desc->d * 2;
  return SEPLLM_OK;
}

extern "C" sepllm_status sepllm_cache_init(const sepllm_cache_desc* desc, void* state,
                                           void* stream_) {
  sepllm_cache_header h;
  sepllm_status st = fill_cache_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (!state || !aligned(state, kAlign)) return SEPLLM_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const size_t words16 = size_t(h.total_bytes) / 16;   // total_bytes is a multiple of 256
  const unsigned blocks = unsigned(std::min<size_t>((words16 + 255) / 256, 1184));
  cache_init_kernel<<<blocks, 256, 0, stream>>>(h, static_cast<uint4*>(state), words16);
  SEPLLM_CUDA_TRY(cudaGetLastError());
  return SEPLLM_OK;
}

static sepllm_status update_impl(const sepllm_cache_desc* desc, void* state, void* Kc, void* Vc,
                                 const int32_t* new_token_ids, const int32_t* sep_ids,
                                 int32_t n_sep, const void* k_new, const void* v_new, void* Kr,
                                 const void* rope_table, bool with_rope, void* stream_) {
  sepllm_cache_header h;
  sepllm_status st = fill_cache_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (!state || !Kc || !Vc || !new_token_ids || !k_new || !v_new) return SEPLLM_INVALID_ARG;
  if (with_rope && (!Kr || !rope_table || !aligned(Kr, 16) || !aligned(rope_table, 16)))
    return SEPLLM_INVALID_ARG;
  if (n_sep < 0 || (n_sep > 0 && !sep_ids)) return SEPLLM_INVALID_ARG;
  if (n_sep > SEPLLM_MAX_SEP_IDS) return SEPLLM_UNSUPPORTED;
  if (!aligned(state, kAlign) || !aligned(Kc, 16) || !aligned(Vc, 16) || !aligned(k_new, 16) ||
      !aligned(v_new, 16))
    return SEPLLM_INVALID_ARG;
  const int max_past = (desc->flags & SEPLLM_CACHE_FIXED_WINDOW) ? 1 : desc->c - desc->a - desc->w;
  if (max_past > kMaxPast || desc->Hkv > 65535) return SEPLLM_UNSUPPORTED;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  SepIds sep;
  sep.n = n_sep;
  for (int k = 0; k < SEPLLM_MAX_SEP_IDS; ++k) sep.id[k] = (k < n_sep) ? sep_ids[k] : -1;
  const size_t smem = size_t(max_past) * sizeof(int16_t);
  auto kernel = with_rope ? cache_update<true> : cache_update<false>;
  if (smem > 40 * 1024)
    SEPLLM_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         int(smem)));
  kernel<<<dim3(desc->B, desc->Hkv), kUpdThreads, smem, stream>>>(
      h, static_cast<uint8_t*>(state), static_cast<__nv_bfloat16*>(Kc),
      static_cast<__nv_bfloat16*>(Vc), static_cast<const __nv_bfloat16*>(k_new),
      static_cast<const __nv_bfloat16*>(v_new), new_token_ids, sep,
      static_cast<__nv_bfloat16*>(Kr), static_cast<const float2*>(rope_table));
  SEPLLM_CUDA_TRY(cudaGetLastError());
  return SEPLLM_OK;
}

extern "C" sepllm_status sepllm_cache_update(const sepllm_cache_desc* desc, void* state, void* Kc,
                                             void* Vc, const int32_t* new_token_ids,
                                             const int32_t* sep_ids, int32_t n_sep,
                                             const void* k_new, const void* v_new,
                                             void* stream_) {
  return update_impl(desc, state, Kc, Vc, new_token_ids, sep_ids, n_sep, k_new, v_new, nullptr,
                     nullptr, false, stream_);
}

extern "C" sepllm_status sepllm_cache_update_rope(const sepllm_cache_desc* desc, void* state,
                                                  void* Kc, void* Vc, void* Kr,
                                                  const void* rope_table,
                                                  const int32_t* new_token_ids,
                                                  const int32_t* sep_ids, int32_t n_sep,
                                                  const void* k_new, const void* v_new,
                                                  void* stream_) {
  return update_impl(desc, state, Kc, Vc, new_token_ids, sep_ids, n_sep, k_new, v_new, Kr,
                     rope_table, true, stream_);
}

extern "C" sepllm_status sepllm_cache_from_prompt(const sepllm_cache_desc* desc,
                                                  const sepllm_index_desc* idesc,
                                                  const void* index, const int32_t* prompt_len,
                                                  const void* K, const void* V, void* state,
                                                  void* Kc, void* Vc, void* Kr,
                                                  const void* rope_table, void* stream_) {
  sepllm_cache_header h;
  sepllm_status st = fill_cache_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  sepllm_index_header ih;
  st = fill_index_header(idesc, &ih);
  if (st != SEPLLM_OK) return st;
  if (!index || !K || !V || !state || !Kc || !Vc) return SEPLLM_INVALID_ARG;
  if (idesc->B != desc->B || idesc->n_init != desc->a) return SEPLLM_INVALID_ARG;
  if (!aligned(index, kAlign) || !aligned(state, kAlign) || !aligned(K, 16) || !aligned(V, 16) ||
      !aligned(Kc, 16) || !aligned(Vc, 16))
    return SEPLLM_INVALID_ARG;
  if ((Kr == nullptr) != (rope_table == nullptr)) return SEPLLM_INVALID_ARG;
  if (Kr && (!aligned(Kr, 16) || !aligned(rope_table, 16))) return SEPLLM_INVALID_ARG;
  if (desc->B > 65535 || desc->Hkv > 65535) return SEPLLM_UNSUPPORTED;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  // the status word starts clean; everything else is written by the plan kernel
  SEPLLM_CUDA_TRY(cudaMemsetAsync(state, 0, sizeof(int32_t), stream));
  prompt_plan<<<desc->B, kPlanThreads, 0, stream>>>(h, static_cast<uint8_t*>(state),
                                                    static_cast<const uint8_t*>(index), ih,
                                                    prompt_len);
  SEPLLM_CUDA_TRY(cudaGetLastError());
  const dim3 grid((h.slots + kCopyRows - 1) / kCopyRows, desc->Hkv, desc->B);
#define SEPLLM_COPY(D, R)                                                                       \
  prompt_copy<D, R><<<grid, kCopyThreads, 0, stream>>>(                                         \
      h, static_cast<const uint8_t*>(state), static_cast<const __nv_bfloat16*>(K),              \
      static_cast<const __nv_bfloat16*>(V), idesc->L, static_cast<__nv_bfloat16*>(Kc),          \
      static_cast<__nv_bfloat16*>(Vc), static_cast<__nv_bfloat16*>(Kr),                         \
      static_cast<const float2*>(rope_table))
  if (desc->d == 128) { if (Kr) SEPLLM_COPY(128, true); else SEPLLM_COPY(128, false); }
  else { if (Kr) SEPLLM_COPY(64, true); else SEPLLM_COPY(64, false); }
#undef SEPLLM_COPY
  SEPLLM_CUDA_TRY(cudaGetLastError());
  return SEPLLM_OK;
}

extern "C" sepllm_status sepllm_decode_workspace_bytes(const sepllm_cache_desc* desc,
                                                       size_t* bytes) {
  sepllm_cache_header h;
  sepllm_status st = fill_cache_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  const int splits = decode_splits(desc);
  const size_t units = size_t(desc->B) * desc->Hq * splits;
  if (bytes) *bytes = kAlign + align_up(units * 2 * sizeof(float)) + align_up(units * desc->d * sizeof(float));
  return SEPLLM_OK;
}

template <int D, bool ROPE, bool WIDE>
static sepllm_status launch_decode(const sepllm_cache_header& h, float scale_log2, const void* q,
                                   const void* state, const void* Kc, const void* Vc, float* ml,
                                   float* acc, int splits, const float2* rope, int32_t* status,
                                   cudaStream_t stream) {
  constexpr int smem = decode_smem_bytes<D>();
  static_assert(smem >= (kDecThreads / 32) * 16 * (8 + D * 4), "partials fit in the stage buffers");
  SEPLLM_CUDA_TRY(cudaFuncSetAttribute(decode_split<D, ROPE, WIDE>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  decode_split<D, ROPE, WIDE><<<dim3(splits, h.desc.Hkv, h.desc.B), kDecThreads, smem, stream>>>(
      h, scale_log2, static_cast<const __nv_bfloat16*>(q), static_cast<const uint8_t*>(state),
      static_cast<const __nv_bfloat16*>(Kc), static_cast<const __nv_bfloat16*>(Vc), ml, acc, splits,
      rope, status);
  return SEPLLM_OK;
}

template <int D>
static sepllm_status dispatch_decode(bool with_rope, bool wide, const sepllm_cache_header& h,
                                     float scale_log2, const void* q, const void* state,
                                     const void* Kc, const void* Vc, float* ml, float* acc,
                                     int splits, const float2* rope, int32_t* status,
                                     cudaStream_t stream) {
#define SEPLLM_DEC(R, W) launch_decode<D, R, W>(h, scale_log2, q, state, Kc, Vc, ml, acc, splits, rope, status, stream)
  if (with_rope) return wide ? SEPLLM_DEC(true, true) : SEPLLM_DEC(true, false);
  return wide ? SEPLLM_DEC(false, true) : SEPLLM_DEC(false, false);
#undef SEPLLM_DEC
}

static sepllm_status decode_impl(const sepllm_cache_desc* desc, float scale, const void* q,
                                 const void* state, const void* Kc, const void* Vc,
                                 const float2* rope, void* o, float* lse, void* workspace,
                                 void* stream_) {
  sepllm_cache_header h;
  sepllm_status st = fill_cache_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (!q || !state || !Kc || !Vc || !o || !workspace) return SEPLLM_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(Kc, 16) || !aligned(Vc, 16) || !aligned(workspace, kAlign) ||
      !aligned(state, kAlign) || !aligned(o, 2))
    return SEPLLM_INVALID_ARG;
  if (desc->B > 65535 || desc->Hkv > 65535) return SEPLLM_UNSUPPORTED;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int splits = decode_splits(desc);
  const size_t units = size_t(desc->B) * desc->Hq * splits;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  // (the decode kernels have no bounded waits and report nothing: the split kernel writes the
  // workspace's status word as OK itself, which saves a memset node per generated token)
  float* ml = reinterpret_cast<float*>(ws + kAlign);
  float* acc = reinterpret_cast<float*>(ws + kAlign + align_up(units * 2 * sizeof(float)));
  if (scale == 0.f) scale = 1.0f / sqrtf(float(desc->d));
  const float scale_log2 = scale * 1.4426950408889634f;
  const bool wide = desc->Hq / desc->Hkv > 8;
  st = (desc->d == 128)
           ? dispatch_decode<128>(rope != nullptr, wide, h, scale_log2, q, state, Kc, Vc, ml, acc, splits, rope,
                                  reinterpret_cast<int32_t*>(ws), stream)
           : dispatch_decode<64>(rope != nullptr, wide, h, scale_log2, q, state, Kc, Vc, ml, acc, splits, rope,
                                 reinterpret_cast<int32_t*>(ws), stream);
  if (st != SEPLLM_OK) return st;
  if (desc->d == 128)
    decode_combine<128><<<dim3(desc->Hq, desc->B), 128, 0, stream>>>(
        h, ml, acc, splits, static_cast<__nv_bfloat16*>(o), lse);
  else
    decode_combine<64><<<dim3(desc->Hq, desc->B), 64, 0, stream>>>(
        h, ml, acc, splits, static_cast<__nv_bfloat16*>(o), lse);
  SEPLLM_CUDA_TRY(cudaGetLastError());
  return SEPLLM_OK;
}

extern "C" sepllm_status sepllm_decode(const sepllm_cache_desc* desc, float scale, const void* q,
                                       const void* state, const void* Kc, const void* Vc, void* o,
                                       float* lse, void* workspace, void* stream_) {
  return decode_impl(desc, scale, q, state, Kc, Vc, nullptr, o, lse, workspace, stream_);
}

extern "C" sepllm_status sepllm_rope_table_bytes(const sepllm_cache_desc* desc, size_t* bytes) {
  sepllm_cache_header h;
  sepllm_status st = fill_cache_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (bytes) *bytes = align_up(size_t(desc->c) * (desc->d / 2) * sizeof(float2));
  return SEPLLM_OK;
}

extern "C" sepllm_status sepllm_rope_table_build(const sepllm_cache_desc* desc, float rope_base,
                                                 void* table, void* stream_) {
  sepllm_cache_header h;
  sepllm_status st = fill_cache_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (!table || !aligned(table, 16) || !(rope_base > 1.f)) return SEPLLM_INVALID_ARG;
  const int n = desc->c * (desc->d / 2);
  rope_table_kernel<<<(n + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream_)>>>(
      static_cast<float2*>(table), desc->c, desc->d / 2, log2f(rope_base));
  SEPLLM_CUDA_TRY(cudaGetLastError());
  return SEPLLM_OK;
}

extern "C" sepllm_status sepllm_decode_rope(const sepllm_cache_desc* desc, float scale,
                                            const void* q, const void* state, const void* Kc,
                                            const void* Vc, const void* rope_table, void* o,
                                            float* lse, void* workspace, void* stream_) {
  if (!rope_table || !aligned(rope_table, 16)) return SEPLLM_INVALID_ARG;
  return decode_impl(desc, scale, q, state, Kc, Vc, static_cast<const float2*>(rope_table), o, lse,
                     workspace, stream_);
}
