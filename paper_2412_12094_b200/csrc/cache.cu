// Streaming KV cache (Section 3.3): update with compaction, and decode attention.
//
// Physical layout per (sequence, kv head): slots = c + s rows of d bf16.
//   [0, a)        Initial Cache, filled once
//   [a, a+s)      ring: Separator Cache (oldest at sep_start)
//   [a+s, c+s)    ring of c-a rows: neighbour run, oldest at win_start; its newest w entries are
//                 the Local Window Cache, the older ones the Past Window Cache
// Decode walks "virtual" entries 0..Size_run-1 = initial, separator (oldest first), neighbour
// (oldest first) and maps each to its slot, so only retained rows are read.
#include "common.cuh"

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
  if (d->Hq / d->Hkv > 8) return SEPLLM_UNSUPPORTED;
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
  if (q.size_init + q.size_sep + size_win == d.c) {
    p.compact = true;
    p.n_past = size_win - d.w;
  }
  return p;
}

constexpr int kUpdThreads = 256;

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

// grid (B, Hkv): K/V movement for one kv head of one sequence.  Reads the state, never writes it.
__global__ void __launch_bounds__(kUpdThreads)
cache_update_kv(sepllm_cache_header h, const uint8_t* __restrict__ state,
                __nv_bfloat16* __restrict__ Kc, __nv_bfloat16* __restrict__ Vc,
                const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new) {
  extern __shared__ int16_t flag_s[];
  __shared__ int warp_buf[32];
  const sepllm_cache_desc d = h.desc;
  const int b = blockIdx.x, hk = blockIdx.y, tid = threadIdx.x;
  CacheView v = cache_view(const_cast<uint8_t*>(state), h);
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
  if (!p.compact || d.s == 0) return;

  const int m = rank_past_separators(v.slot_is_sep + size_t(b) * h.slots, q, d, p.n_past, flag_s,
                                     warp_buf);
  const int drop = max(0, q.size_sep + m - d.s);
  const int ring = d.c - d.a, wbase = d.a + d.s;
  // one half-warp (16 lanes x 16 bytes = 256 bytes) moves a K row, the other the V row when d=128;
  // generic: `vec` lanes per row
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

// grid (B): per-slot metadata and the sequence record.  Runs after cache_update_kv.
__global__ void __launch_bounds__(kUpdThreads)
cache_update_state(sepllm_cache_header h, uint8_t* __restrict__ state,
                   const int32_t* __restrict__ new_token_ids, SepIds sep) {
  extern __shared__ int16_t flag_s[];
  __shared__ int warp_buf[32];
  const sepllm_cache_desc d = h.desc;
  const int b = blockIdx.x, tid = threadIdx.x;
  CacheView v = cache_view(state, h);
  const sepllm_cache_seq q = v.seq[b];
  const UpdatePlan p = plan_update(q, d);
  int64_t* pos_b = v.slot_pos + size_t(b) * h.slots;
  uint8_t* sep_b = v.slot_is_sep + size_t(b) * h.slots;
  const bool f = is_separator(new_token_ids[b], sep);
  __syncthreads();  // every thread holds the old record before it changes
  if (tid == 0) {
    pos_b[p.append_slot] = q.next_pos;
    sep_b[p.append_slot] = uint8_t(f);
  }
  sepllm_cache_seq nq = q;
  nq.next_pos = q.next_pos + 1;
  if (q.size_init < d.a) nq.size_init = q.size_init + 1;
  else nq.size_win = q.size_win + 1;

  if (p.compact) {
    int m = 0, drop = 0;
    if (d.s > 0) {
      m = rank_past_separators(sep_b, q, d, p.n_past, flag_s, warp_buf);
      drop = max(0, q.size_sep + m - d.s);
      const int ring = d.c - d.a, wbase = d.a + d.s;
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
      nq.sep_start = (q.sep_start + drop) % d.s;
      nq.size_sep = q.size_sep + m - drop;
    }
    nq.win_start = (q.win_start + p.n_past) % (d.c - d.a);
    nq.size_win = d.w;
    nq.compactions = q.compactions + 1;
  }
  if (tid == 0) v.seq[b] = nq;
}

// ---------------------------------------------------------------------------
// Decode: one query per sequence over the retained entries
// ---------------------------------------------------------------------------
constexpr int kDecThreads = 128;

__device__ __forceinline__ int virtual_to_slot(int v, const sepllm_cache_seq& q,
                                               const sepllm_cache_desc& d) {
  if (v < q.size_init) return v;
  v -= q.size_init;
  if (v < q.size_sep) return d.a + (q.sep_start + v) % d.s;
  v -= q.size_sep;
  return d.a + d.s + (q.win_start + v) % (d.c - d.a);
}

// grid (splits, Hkv, B).  Each warp takes rows of its split in turn; a row of D bf16 is read by
// D/8 lanes with one 16-byte load each, so a warp covers 32/(D/8) rows per step.  The G query
// heads sharing the kv head are handled together so K and V are read once.
template <int D, int G>
__global__ void __launch_bounds__(kDecThreads)
decode_split(sepllm_cache_header h, float scale_log2, const __nv_bfloat16* __restrict__ q_in,
             const uint8_t* __restrict__ state, const __nv_bfloat16* __restrict__ Kc,
             const __nv_bfloat16* __restrict__ Vc, float* __restrict__ part_ml,
             float* __restrict__ part_acc, int splits) {
  constexpr int LPR = D / 8;        // lanes per row
  constexpr int RPW = 32 / LPR;     // rows per warp step
  constexpr int NW = kDecThreads / 32;
  const sepllm_cache_desc d = h.desc;
  const int split = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int sub = lane / LPR, l = lane % LPR;
  CacheView cv = cache_view(const_cast<uint8_t*>(state), h);
  const sepllm_cache_seq sq = cv.seq[b];
  const int size_run = sq.size_init + sq.size_sep + sq.size_win;
  const int per = (size_run + splits - 1) / splits;
  const int v0 = split * per, v1 = min(size_run, v0 + per);

  // this lane's 8 elements of each of the G queries, pre-scaled to log2 units
  float qf[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const uint4 raw = *reinterpret_cast<const uint4*>(
        q_in + (size_t(b) * d.Hq + hk * G + g) * D + l * 8);
    const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f2 = __bfloat1622float2(p2[e]);
      qf[g][2 * e] = f2.x * scale_log2;
      qf[g][2 * e + 1] = f2.y * scale_log2;
    }
  }
  float m[G], lsum[G], acc[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m[g] = -INFINITY;
    lsum[g] = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[g][e] = 0.f;
  }
  const size_t plane = (size_t(b) * d.Hkv + hk) * h.slots * D;
  // Every lane of the warp takes the same number of trips (the shuffles below need all 32
  // lanes); a sub-row past the end of the split reloads the last row and is not accumulated.
  for (int base = v0 + wid * RPW; base < v1; base += NW * RPW) {
    const int vrow = base + sub;
    const bool valid = vrow < v1;
    const int slot = virtual_to_slot(valid ? vrow : v1 - 1, sq, d);
    const uint4 kraw = *reinterpret_cast<const uint4*>(Kc + plane + size_t(slot) * D + l * 8);
    const uint4 vraw = *reinterpret_cast<const uint4*>(Vc + plane + size_t(slot) * D + l * 8);
    const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&kraw);
    const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&vraw);
    float kf[8], vf[8];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 a2 = __bfloat1622float2(k2[e]);
      const float2 b2 = __bfloat1622float2(v2[e]);
      kf[2 * e] = a2.x; kf[2 * e + 1] = a2.y;
      vf[2 * e] = b2.x; vf[2 * e + 1] = b2.y;
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float s = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) s = fmaf(qf[g][e], kf[e], s);
#pragma unroll
      for (int o = LPR / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (valid) {
        const float mn = fmaxf(m[g], s);
        const float corr = ex2(m[g] - mn);
        const float pexp = ex2(s - mn);
        m[g] = mn;
        lsum[g] = lsum[g] * corr + pexp;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[g][e] = fmaf(acc[g][e], corr, pexp * vf[e]);
      }
    }
  }

  // combine the RPW sub-rows of the warp, then the NW warps, through shared memory
  __shared__ float sm_m[NW * RPW][G];
  __shared__ float sm_l[NW * RPW][G];
  __shared__ float sm_acc[NW * RPW][G][D];
  const int slot_id = wid * RPW + sub;
#pragma unroll
  for (int g = 0; g < G; ++g) {
    if (l == 0) { sm_m[slot_id][g] = m[g]; sm_l[slot_id][g] = lsum[g]; }
#pragma unroll
    for (int e = 0; e < 8; ++e) sm_acc[slot_id][g][l * 8 + e] = acc[g][e];
  }
  __syncthreads();
  for (int idx = tid; idx < G * D; idx += kDecThreads) {
    const int g = idx / D, e = idx % D;
    float mm = -INFINITY;
#pragma unroll
    for (int r = 0; r < NW * RPW; ++r) mm = fmaxf(mm, sm_m[r][g]);
    float ll = 0.f, aa = 0.f;
#pragma unroll
    for (int r = 0; r < NW * RPW; ++r) {
      const float sc = (sm_m[r][g] == -INFINITY) ? 0.f : ex2(sm_m[r][g] - mm);
      ll += sm_l[r][g] * sc;
      aa += sm_acc[r][g][e] * sc;
    }
    const size_t u = ((size_t(b) * d.Hq + hk * G + g) * splits + split);
    part_acc[u * D + e] = aa;
    if (e == 0) { part_ml[u * 2] = mm; part_ml[u * 2 + 1] = ll; }
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

static int decode_splits(const sepllm_cache_desc* d) {
  // enough CTAs for several per SM, at least ~128 rows each
  const int units = d->B * d->Hkv;
  int s = (148 * 8 + units - 1) / units;
  const int max_by_rows = (d->c + 127) / 128;
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
  SEPLLM_CUDA_TRY(cudaMemsetAsync(state, 0, size_t(h.total_bytes), stream));
  SEPLLM_CUDA_TRY(cudaMemcpyAsync(state, &h, sizeof(h), cudaMemcpyHostToDevice, stream));
  // the header lives on this call's stack: make sure the copy has read it
  SEPLLM_CUDA_TRY(cudaStreamSynchronize(stream));
  return SEPLLM_OK;
}

extern "C" sepllm_status sepllm_cache_update(const sepllm_cache_desc* desc, void* state, void* Kc,
                                             void* Vc, const int32_t* new_token_ids,
                                             const int32_t* sep_ids, int32_t n_sep,
                                             const void* k_new, const void* v_new,
                                             void* stream_) {
  sepllm_cache_header h;
  sepllm_status st = fill_cache_header(desc, &h);
  if (st != SEPLLM_OK) return st;
  if (!state || !Kc || !Vc || !new_token_ids || !k_new || !v_new) return SEPLLM_INVALID_ARG;
  if (n_sep < 0 || (n_sep > 0 && !sep_ids)) return SEPLLM_INVALID_ARG;
  if (n_sep > SEPLLM_MAX_SEP_IDS) return SEPLLM_UNSUPPORTED;
  if (!aligned(state, kAlign) || !aligned(Kc, 16) || !aligned(Vc, 16) || !aligned(k_new, 16) ||
      !aligned(v_new, 16))
    return SEPLLM_INVALID_ARG;
  const int max_past = desc->c - desc->a - desc->w;
  if (max_past > kMaxPast || desc->Hkv > 65535) return SEPLLM_UNSUPPORTED;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  SepIds sep;
  sep.n = n_sep;
  for (int k = 0; k < SEPLLM_MAX_SEP_IDS; ++k) sep.id[k] = (k < n_sep) ? sep_ids[k] : -1;
  const size_t smem = size_t(max_past) * sizeof(int16_t);
  if (smem > 40 * 1024) {
    SEPLLM_CUDA_TRY(cudaFuncSetAttribute(cache_update_kv,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    SEPLLM_CUDA_TRY(cudaFuncSetAttribute(cache_update_state,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
  }
  cache_update_kv<<<dim3(desc->B, desc->Hkv), kUpdThreads, smem, stream>>>(
      h, static_cast<const uint8_t*>(state), static_cast<__nv_bfloat16*>(Kc),
      static_cast<__nv_bfloat16*>(Vc), static_cast<const __nv_bfloat16*>(k_new),
      static_cast<const __nv_bfloat16*>(v_new));
  cache_update_state<<<desc->B, kUpdThreads, smem, stream>>>(h, static_cast<uint8_t*>(state),
                                                            new_token_ids, sep);
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

template <int D, int G>
static void launch_decode(const sepllm_cache_header& h, float scale_log2, const void* q,
                          const void* state, const void* Kc, const void* Vc, float* ml, float* acc,
                          int splits, cudaStream_t stream) {
  decode_split<D, G><<<dim3(splits, h.desc.Hkv, h.desc.B), kDecThreads, 0, stream>>>(
      h, scale_log2, static_cast<const __nv_bfloat16*>(q), static_cast<const uint8_t*>(state),
      static_cast<const __nv_bfloat16*>(Kc), static_cast<const __nv_bfloat16*>(Vc), ml, acc,
      splits);
}

extern "C" sepllm_status sepllm_decode(const sepllm_cache_desc* desc, float scale, const void* q,
                                       const void* state, const void* Kc, const void* Vc, void* o,
                                       float* lse, void* workspace, void* stream_) {
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
  float* ml = reinterpret_cast<float*>(ws + kAlign);
  float* acc = reinterpret_cast<float*>(ws + kAlign + align_up(units * 2 * sizeof(float)));
  if (scale == 0.f) scale = 1.0f / sqrtf(float(desc->d));
  const float scale_log2 = scale * 1.4426950408889634f;
  const int G = desc->Hq / desc->Hkv;
#define SEPLLM_DEC(DD, GG)                                                                      \
  if (desc->d == DD && G == GG) {                                                               \
    launch_decode<DD, GG>(h, scale_log2, q, state, Kc, Vc, ml, acc, splits, stream);           \
  } else
  SEPLLM_DEC(128, 1) SEPLLM_DEC(128, 2) SEPLLM_DEC(128, 4) SEPLLM_DEC(128, 8)
  SEPLLM_DEC(64, 1) SEPLLM_DEC(64, 2) SEPLLM_DEC(64, 4) SEPLLM_DEC(64, 8)
  { return SEPLLM_UNSUPPORTED; }
#undef SEPLLM_DEC
  if (desc->d == 128)
    decode_combine<128><<<dim3(desc->Hq, desc->B), 128, 0, stream>>>(
        h, ml, acc, splits, static_cast<__nv_bfloat16*>(o), lse);
  else
    decode_combine<64><<<dim3(desc->Hq, desc->B), 64, 0, stream>>>(
        h, ml, acc, splits, static_cast<__nv_bfloat16*>(o), lse);
  SEPLLM_CUDA_TRY(cudaGetLastError());
  return SEPLLM_OK;
}
