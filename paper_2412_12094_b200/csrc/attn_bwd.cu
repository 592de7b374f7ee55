// Backward of separator-masked attention for sm_100a.
//
// With P = softmax(S) (recomputed from LSE), dP = dO V^T, Delta_i = sum(dO_i * O_i):
//   dS = P * (dP - Delta);  dQ = dS K * scale;  dK = dS^T Q * scale;  dV = P^T dO.
// Three passes, none using floating-point atomics, so results are deterministic:
//   bwd_delta     Delta for every query row.
//   bwd_dq        query-tile stationary: walks the same side + window key tiles as the forward
//                 and accumulates dQ in tensor memory.
//   bwd_dkv<SIDE> key-tile stationary: one CTA owns 128 keys (a tile of the side buffer, or a tile
//                 of K/V for the neighbour window), walks every query tile that keeps any of them
//                 and every query head of the GQA group, and accumulates dK, dV in tensor memory.
//                 A separator far behind many queries is therefore summed inside one CTA instead
//                 of being the target of contended atomics.  The side pass runs first and leaves
//                 fp32 partial rows; the window pass adds them to the rows of the same tokens
//                 before rounding once to the output type.
#include <algorithm>

#include "attn_common.cuh"

namespace sepllm {

constexpr float kLog2e = 1.4426950408889634f;

// ---------------------------------------------------------------------------
// Row statistics: (LSE in log2 units, Delta) per query row
// ---------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256)
bwd_delta(const __nv_bfloat16* __restrict__ dO, const __nv_bfloat16* __restrict__ O,
          const float* __restrict__ LSE, float2* __restrict__ stats, size_t rows, int d) {
  constexpr int LPR = D / 8;
  const size_t r = (size_t(blockIdx.x) * 256 + threadIdx.x) / LPR;
  const int l = threadIdx.x % LPR;
  float s = 0.f;
  if (r < rows && l * 8 < d) {   // rows of d <= D elements
    const uint4 a = *reinterpret_cast<const uint4*>(dO + r * d + l * 8);
    const uint4 b = *reinterpret_cast<const uint4*>(O + r * d + l * 8);
    const __nv_bfloat162* a2 = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* b2 = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 x = __bfloat1622float2(a2[e]), y = __bfloat1622float2(b2[e]);
      s = fmaf(x.x, y.x, s);
      s = fmaf(x.y, y.y, s);
    }
  }
#pragma unroll
  for (int o = LPR / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (r < rows && l == 0) stats[r] = make_float2(LSE[r] * kLog2e, s);
}

struct BwdParams {
  const int32_t* cnt;        // [B][L+1]
  const int32_t* lim;        // [B][L]
  const int32_t* side_pos;   // [B][side_cap]
  const int32_t* n_side;     // [B]
  const int32_t* tile_meta;  // [B][T][8]
  const int32_t* seq_len;    // [B]
  const sepllm_index_header* index_header;   // on the device (its `packed` word is read there)
  const int32_t* doc_start;  // [B][L]   (packed index only)
  const int32_t* doc_end;    // [B][L]
  const float2* stats;       // [B][Hq][L] (LSE * log2 e, Delta)
  float* dKs;                // [split][B][Hkv][cap_pad][D] fp32 side partials
  float* dVs;
  void* dQ;
  void* dK;
  void* dV;
  int32_t* status;
  int B, L, T, Hq, Hkv, n_neighbor, side_cap, cap_pad, grad_fp32, split, pair_heads;
  int d;                     // row length of Q, K, V, dO and the gradients in memory (<= D)
  float scale, scale_log2;
};

// n_cols (a multiple of 8): how many of the 32 values lie inside the row.
__device__ __forceinline__ void store_row_chunk32(void* base, size_t elem_off, int fp32,
                                                  const float (&v)[32], int n_cols = 32) {
  if (fp32) {
    float4* dst = reinterpret_cast<float4*>(static_cast<float*>(base) + elem_off);
#pragma unroll
    for (int q = 0; q < 8; ++q)
      if (4 * q < n_cols) dst[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
  } else {
    uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(base) + elem_off);
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (8 * q < n_cols)
        dst[q] = make_uint4(pack_bf16(v[8 * q], v[8 * q + 1]), pack_bf16(v[8 * q + 2], v[8 * q + 3]),
                            pack_bf16(v[8 * q + 4], v[8 * q + 5]), pack_bf16(v[8 * q + 6], v[8 * q + 7]));
  }
}

constexpr int kBwdThreads = 384;
constexpr int kFar = 0x3fffffff;                // "never" / "unbounded" for column ranges

// ---------------------------------------------------------------------------
// dQ: query-tile stationary
// ---------------------------------------------------------------------------
// One CTA owns one query tile of one head.  Shared-memory bandwidth and the near-empty MMA queue
// are what bound these kernels, so the stationary operands Q and dO are kept in tensor memory
// (packed bf16, written once by the arithmetic threads straight from global memory), only the
// streamed K / V tiles pass through shared memory, and every MMA is 128 wide:
//   warp 0      TMA producer: [K | V] tiles of 128 keys through a ring
//   warp 1      MMA issuer:   S = Q K^T, dP = dO V^T (A from tensor memory), dQ += dS K
//   warps 4-11  dS = P (dP - Delta): thread = query row, warpgroup u takes key columns
//               [64u, 64u+64).  S is released as soon as it has been loaded so that the next
//               tile's S MMAs run under this tile's arithmetic; dS goes over the dP columns.
template <int D>
struct DqCfg {
  static constexpr int NB = D / 64;
  static constexpr int NST = 3;
  static constexpr uint32_t kTile = NB * kTileBlockBytes;   // one 128-key tile of K or V
  static constexpr uint32_t kStage = 2 * kTile;
  static constexpr uint32_t kKV = 0;
  static constexpr uint32_t kBar = kKV + NST * kStage;
  static constexpr uint32_t kTotal = kBar + 512;
  static constexpr uint32_t kRequest = (kTotal + 1024 > 116 * 1024) ? kTotal + 1024 : 116 * 1024;
  // tensor-memory columns
  static constexpr uint32_t kQt = 0, kdOt = 64, kS = 128, kdP = 256, kdQ = 384;
};

// One unit of work of the dQ kernel: a query tile of one head.
struct DqItem {
  int t, kv_plane, q_plane, b, sbase, ns, wlo, n_tiles;   // key tiles: side [sbase, sbase + ns), window from wlo
  SlotGeom g;
};
// Items are numbered tile-major (longest tiles first), heads x batch minor, so that the heads of
// a GQA group work on the same K/V tiles at the same time.
__device__ __forceinline__ DqItem dq_item(const BwdParams& p, const DocView& dv, int w) {
  const int hb = p.Hq * p.B;
  const int x = w % hb;
  DqItem it;
  it.b = x / p.Hq;
  const int hq = x % p.Hq;
  it.t = p.T - 1 - w / hb;
  const SlotGeom g = load_slot(p.tile_meta, p.seq_len, it.b, p.T, it.t, hq, p.cap_pad / kBN, dv, p.L,
                               p.n_neighbor);
  it.kv_plane = it.b * p.Hkv + hq / (p.Hq / p.Hkv);
  it.q_plane = it.b * p.Hq + hq;
  it.sbase = (g.t >= 0) ? g.s0 : 0;
  it.ns = max(0, g.ns - it.sbase);
  it.wlo = g.wlo;
  it.n_tiles = (g.t >= 0) ? it.ns + (g.whi - g.wlo) : 0;   // 0: a tile of padding, skipped by every role
  it.g = g;
  return it;
}

// Persistent: one CTA per SM walks items w = blockIdx.x, blockIdx.x + gridDim.x, ...  Stage and
// barrier phases run on a tile count that continues across items; the next item's Q and dO go
// into tensor memory as soon as the current item's last S / dP MMAs are complete, and its first
// MMAs run while the current item's dQ is still being stored.
// PACKED: the index holds document bounds.  There is one kernel per body (see bwd_dq_kernel);
// without the bounds every test for them is compiled out (as
// run-time tests they cost this kernel, which decodes an item in every role, 8 % of its time).
template <int D, bool PACKED>
__device__ __forceinline__ void
bwd_dq_body(const CUtensorMap& mapK, const CUtensorMap& mapV, const CUtensorMap& mapKs,
            const CUtensorMap& mapVs, const __nv_bfloat16* __restrict__ Qg,
            const __nv_bfloat16* __restrict__ dOg, const BwdParams& p, const int n_items) {
  using C = DqCfg<D>;
  constexpr int NB = C::NB, NST = C::NST;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~uintptr_t(1023));
  uint8_t* sKV = smem + C::kKV;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kBar);
  uint64_t* bar_qdo = bars;            //       Q and dO of an item written to tensor memory (8 warps)
  uint64_t* bar_acc = bars + 1;        //       every MMA of an item complete
  uint64_t* bar_s = bars + 2;          //       S of a tile complete
  uint64_t* bar_sl = bars + 3;         //       S of a tile loaded into registers (8 warps)
  uint64_t* bar_ds = bars + 4;         //       dS of a tile written (8 warps)
  uint64_t* bar_dp = bars + 5;         //       dP of a tile complete
  uint64_t* bar_dqf = bars + 6;        //       dQ of an item read out of tensor memory (8 warps)
  uint64_t* bar_f = bars + 7;          // [NST] stage full
  uint64_t* bar_e = bar_f + NST;       // [NST] stage free (its dQ MMAs are complete; one arithmetic thread arrives)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 7 + 2 * NST);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    mbar_init(bar_qdo, 8);
    mbar_init(bar_acc, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_dp, 1);
    mbar_init(bar_sl, 8);
    mbar_init(bar_ds, 8);
    mbar_init(bar_dqf, 8);
    for (int i = 0; i < NST; ++i) { mbar_init(bar_f + i, 1); mbar_init(bar_e + i, 1); }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  const DocView dv = PACKED ? DocView{p.cnt, p.doc_start, p.doc_end} : DocView{nullptr, nullptr, nullptr};
  bool ok = true;
  auto wait = [&](uint64_t* bar, uint32_t parity) {
    if (!mbar_wait(bar, parity, abort_flag)) {
      if (ok) set_status(p.status, SEPLLM_TIMEOUT);
      ok = false;
    }
  };

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 104;");
    if (warp == 0 && lane == 0) {
      // ---------------- TMA producer ----------------
      int tb = 0;  // tiles before this item
      for (int w = blockIdx.x; w < n_items; w += gridDim.x) {
        const DqItem it = dq_item(p, dv, w);   // (an empty item has no tiles)
        for (int j = 0; j < it.n_tiles; ++j) {
          const bool side = j < it.ns;
          const int y = side ? (it.sbase + j) * kBN : (it.wlo + (j - it.ns)) * kBN;
          const int gi = tb + j, st = gi % NST;
          if (gi >= NST) wait(bar_e + st, (gi / NST - 1) & 1);
          mbar_expect_tx(bar_f + st, C::kStage);
          uint8_t* dst = sKV + st * C::kStage;
          for (int nb = 0; nb < NB; ++nb) {
            tma_load_3d(dst + nb * kTileBlockBytes, side ? &mapKs : &mapK, bar_f + st, nb * 64, y,
                        it.kv_plane);
            tma_load_3d(dst + C::kTile + nb * kTileBlockBytes, side ? &mapVs : &mapV, bar_f + st,
                        nb * 64, y, it.kv_plane);
          }
        }
        tb += it.n_tiles;
      }
    } else if (warp == 1 && lane == 0) {
      // ---------------- MMA issuer ----------------
      constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);
      constexpr uint32_t idesc_dq = make_idesc_bf16(128, D, 0, 1);
      const uint32_t k_lo0 = desc_lo(smem_u32(sKV), 16);                // K as the K-major B of S
      const uint32_t kt_lo0 = desc_lo(smem_u32(sKV), kTileBlockBytes);  // K as the MN-major B of dQ
      // The issuing thread's own scalar instructions sit between the MMAs of consecutive groups
      // (one warp issues a dependent instruction every few cycles, and the tensor pipe holds next
      // to no queue), so the loop carries the ring stage and the barrier parities along instead of
      // dividing tile counters.
      auto issue_s = [&](int st) {
        const uint32_t k_lo = k_lo0 + st * (C::kStage >> 4);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          umma_ts_lo(tmem + C::kS, tmem + C::kQt + k * 8, k_lo + kmajor_step(k, kTileBlockBytes),
                     idesc_s, k > 0);
        tc_commit(bar_s);
      };
      auto issue_dp = [&](int st) {
        const uint32_t v_lo = k_lo0 + st * (C::kStage >> 4) + (C::kTile >> 4);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          umma_ts_lo(tmem + C::kdP, tmem + C::kdOt + k * 8, v_lo + kmajor_step(k, kTileBlockBytes),
                     idesc_s, k > 0);
        tc_commit(bar_dp);
      };
      int ino = 0;
      int st = 0;            // ring stage of the current tile
      uint32_t fpar = 0;     // parity of that stage's "full" barrier
      uint32_t gpar = 0;     // parity of the per-tile barriers (tile counter & 1)
      for (int w = blockIdx.x; w < n_items; w += gridDim.x) {
        const int n_tiles = dq_item(p, dv, w).n_tiles;
        if (n_tiles == 0) continue;
        wait(bar_qdo, ino & 1);
        wait(bar_f + st, fpar);
        tc_fence_after();
        issue_s(st);
        issue_dp(st);
        for (int j = 0; j < n_tiles; ++j) {
          int st1 = st + 1;
          uint32_t fpar1 = fpar;
          if (st1 == NST) { st1 = 0; fpar1 ^= 1u; }
          if (j + 1 < n_tiles) {
            // S of the next tile as soon as this tile's S has been read out
            wait(bar_f + st1, fpar1);
            wait(bar_sl, gpar);
            tc_fence_after();
            issue_s(st1);
          }
          wait(bar_ds, gpar);
          if (j == 0 && ino > 0) wait(bar_dqf, (ino - 1) & 1);  // the previous item's dQ is stored
          tc_fence_after();
          // dS of keys [64u, 64u+64) sits in columns 64u .. 64u+31 of the dP range
          const uint32_t kt_lo = kt_lo0 + st * (C::kStage >> 4);
#pragma unroll
          for (int k = 0; k < kBN / 16; ++k)
            umma_ts_lo(tmem + C::kdQ, tmem + C::kdP + (k >> 2) * 64 + (k & 3) * 8,
                       kt_lo + mnmajor_step(k), idesc_dq, (j > 0 || k > 0));
          // (the stage is reported free by an arithmetic warp once it sees the next dP complete:
          // a commit here would cost this thread about 90 cycles of tensor-pipe idle time)
          if (j + 1 < n_tiles) issue_dp(st1);
          st = st1;
          fpar = fpar1;
          gpar ^= 1u;
        }
        tc_commit(bar_acc);
        ++ino;
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 200;");
    const int u = (warp >= 8) ? 1 : 0;
    const int r = tid & 127;
    const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_base + C::kS + u * 64;
    const uint32_t tdP = tmem + lane_base + C::kdP + u * 64;
    // Q (warps 4-7) or dO (warps 8-11) row of an item into tensor memory
    auto load_qdo = [&](const DqItem& it) {
      const int row = it.t * kBM + r;
      const bool row_ok = row < p.L;
      const uint4* src = reinterpret_cast<const uint4*>((u ? dOg : Qg) +
                                                        (size_t(it.q_plane) * p.L + row) * p.d);
      const uint32_t dst = tmem + lane_base + (u ? C::kdOt : C::kQt);
#pragma unroll
      for (int c = 0; c < D / 64; ++c) {
        uint32_t w[32];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const uint4 v = (row_ok && (c * 8 + q) * 8 < p.d) ? src[c * 8 + q] : make_uint4(0, 0, 0, 0);
          w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
        }
        tmem_st32(dst + c * 32, w);
      }
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive_warp(bar_qdo);
    };
    int tb = 0, ino = 0;
    // the next item of this CTA that has work, from w on
    auto next_item = [&](int w) {
      while (w < n_items && dq_item(p, dv, w).n_tiles == 0) w += gridDim.x;
      return w;
    };
    int w = next_item(blockIdx.x);
    if (w < n_items) load_qdo(dq_item(p, dv, w));
    for (; w < n_items; ++ino) {
      const DqItem it = dq_item(p, dv, w);
      const int w_next = next_item(w + gridDim.x);
      // The next item's Q / dO row is loaded at the hand-over between items, where the tensor pipe
      // waits for it: ask for its lines now, a whole item ahead, so that the load finds them in L2.
      if (w_next < n_items) {
        const DqItem nx = dq_item(p, dv, w_next);
        const int nrow = nx.t * kBM + r;
        if (nrow < p.L) {
          const char* a = reinterpret_cast<const char*>((u ? dOg : Qg) + (size_t(nx.q_plane) * p.L + nrow) * p.d);
          for (int off = 0; off < p.d * 2; off += 128)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(a + off));
        }
      }
      const int t = it.t, ns = it.ns;
      const int row = t * kBM + r;
      const bool row_ok = row < p.L;
      // ---------------- dS: warpgroup u takes key columns [64u, 64u+64) of every tile ---------
      const RowGeom rg = row_geom(p.lim, dv, it.b, p.L, row, p.n_neighbor, p.side_cap);
      const float2 stt = row_ok ? p.stats[size_t(it.q_plane) * p.L + row] : make_float2(INFINITY, 0.f);
      const float neg_lse2 = -stt.x, delta_i = stt.y;
      for (int j = 0; j < it.n_tiles; ++j) {
        const int gi = tb + j;
        const bool side = j < ns;
        int c_lo, c_hi;
        bool need_mask;
        key_range(side, side ? it.sbase + j : it.wlo + (j - ns), it.g, row, rg, c_lo, c_hi, need_mask);
        // phase A (needs S only; runs under the previous tile's dQ and this tile's dP MMAs):
        // P = exp2(S * scale - LSE), kept in registers
        wait(bar_s, gi & 1);
        tc_fence_after();
        uint32_t sv[2][32];
        tmem_ld32(tS, sv[0]);
        tmem_ld32(tS + 32, sv[1]);
        tmem_ld_wait();
        tc_fence_before();
        mbar_arrive_warp(bar_sl);  // the S columns may be overwritten from here on
        // packed fp32 pairs: one multiply-add instruction per two scores
        const unsigned long long scale2 = pack_f32x2(p.scale_log2, p.scale_log2);
        const unsigned long long nlse2 = pack_f32x2(neg_lse2, neg_lse2);
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float2 a = unpack_f32x2(fma_f32x2(
                pack_f32x2(__uint_as_float(sv[c][e]), __uint_as_float(sv[c][e + 1])), scale2, nlse2));
            float p0 = ex2(a.x), p1 = ex2(a.y);
            if (need_mask) {
              const int col = u * 64 + c * 32 + e;
              p0 = (col >= c_lo && col < c_hi) ? p0 : 0.f;
              p1 = (col + 1 >= c_lo && col + 1 < c_hi) ? p1 : 0.f;
            }
            sv[c][e] = __float_as_uint(p0);
            sv[c][e + 1] = __float_as_uint(p1);
          }
        // phase B: dS = P (dP - Delta)
        wait(bar_dp, gi & 1);
        tc_fence_after();
        // MMAs complete in issue order and dQ of the tile before this one (of this item or the
        // last of the previous one) was issued before this dP: its K/V stage is free
        if (tid == 128 && gi > 0) mbar_arrive(bar_e + (gi - 1) % NST);
        uint32_t pk[32];
        const unsigned long long ndelta2 = pack_f32x2(-delta_i, -delta_i);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t dp[32];
          tmem_ld32(tdP + c * 32, dp);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const unsigned long long t2 = add_f32x2(
                pack_f32x2(__uint_as_float(dp[e]), __uint_as_float(dp[e + 1])), ndelta2);
            const float2 ds = unpack_f32x2(mul_f32x2(
                pack_f32x2(__uint_as_float(sv[c][e]), __uint_as_float(sv[c][e + 1])), t2));
            pk[c * 16 + (e >> 1)] = pack_bf16(ds.x, ds.y);
          }
        }
        // packed dS over the first half of this thread's own dP columns
        tmem_st32(tdP, pk);
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive_warp(bar_ds);
      }
      tb += it.n_tiles;
      // Every S and dP MMA of this item is complete (the last dP was waited for), so Q and dO of
      // the next item can go into tensor memory while this item's last dQ MMAs run.
      if (w_next < n_items) load_qdo(dq_item(p, dv, w_next));
      // ---------------- epilogue: each warpgroup stores half of the row ----------------
      wait(bar_acc, ino & 1);
      tc_fence_after();
      const uint32_t t_acc = tmem + lane_base + C::kdQ + u * (D / 2);
#pragma unroll
      for (int c = 0; c < D / 64; ++c) {
        uint32_t rr[32];
        tmem_ld32(t_acc + c * 32, rr);
        tmem_ld_wait();
        if (c == D / 64 - 1) {  // dQ is in registers: the next item may start accumulating
          tc_fence_before();
          mbar_arrive_warp(bar_dqf);
        }
        if (row_ok) {
          float v[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(rr[e]) * p.scale;
          const int col = u * (D / 2) + c * 32;
          store_row_chunk32(p.dQ, (size_t(it.q_plane) * p.L + row) * p.d + col, p.grad_fp32, v,
                            p.d - col);
        }
      }
      w = w_next;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

// Both instances are launched, one after the other; the one that does not match the index
// header's `packed` word returns at once (the host cannot read that word without a
// synchronisation).  One kernel holding both bodies ran the common one 3 % slower than it runs
// alone, and a called (not inlined) second body 17 % slower; an empty launch costs 2-3 us.
template <int D, bool PACKED>
__global__ void __launch_bounds__(kBwdThreads, 1)
bwd_dq_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
              const __grid_constant__ CUtensorMap mapKs, const __grid_constant__ CUtensorMap mapVs,
              const __nv_bfloat16* __restrict__ Qg, const __nv_bfloat16* __restrict__ dOg,
              const BwdParams p, const int n_items) {
  if ((p.index_header->packed != 0) != PACKED) return;
  bwd_dq_body<D, PACKED>(mapK, mapV, mapKs, mapVs, Qg, dOg, p, n_items);
}

// ---------------------------------------------------------------------------
// dK, dV: key-tile stationary
// ---------------------------------------------------------------------------
// One CTA owns 128 keys and streams the query tiles (128 rows of one query head per iteration)
// that keep any of them:
//   warp 0      TMA producer (K, V once; then Q and dO per iteration through rings of their own)
//   warp 1      MMA issuer:  S^T = K Q^T, dP^T = V dO^T (128 wide), then dV += P^T dO and
//               dK += dS^T Q with A taken from tensor memory
//   warps 2-3   load the 128 (LSE, Delta) pairs of the iteration into shared memory
//   warps 4-11  P^T and dS^T (thread = key row); warpgroup u takes query columns [64u, 64u+64).
//               S^T is released as soon as it has been loaded, so the next iteration's S^T MMAs
//               run under this iteration's arithmetic; P^T and dS^T go, packed, over the two
//               halves of the thread's own dP^T columns.
template <int D>
struct DkvCfg {
  static constexpr int NB = D / 64;
  // Q is needed one iteration earlier than dO (S^T runs under the previous iteration's
  // arithmetic), so it gets the deeper ring; a tile takes about a microsecond to arrive.
  static constexpr int NSQ = 3, NSO = 2;
  static constexpr uint32_t kTile = NB * kTileBlockBytes;
  static constexpr uint32_t kK = 0;
  static constexpr uint32_t kV = kK + kTile;
  static constexpr uint32_t kQ = kV + kTile;                 // NSQ x Q
  static constexpr uint32_t kdO = kQ + NSQ * kTile;          // NSO x dO
  static constexpr uint32_t kStat = kdO + NSO * kTile;       // 128 float2, one iteration at a time
  static constexpr uint32_t kBar = kStat + 128 * 8;
  static constexpr uint32_t kTotal = kBar + 512;
  static constexpr uint32_t kRequest = (kTotal + 1024 > 116 * 1024) ? kTotal + 1024 : 116 * 1024;
  static_assert(kRequest <= 227 * 1024, "shared memory budget");
  // tensor-memory columns
  static constexpr uint32_t kdV = 0, kdK = D, kST = 256, kdPT = 384;
};

template <int D, bool SIDE>
__global__ void __launch_bounds__(kBwdThreads, 1)
bwd_dkv_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapdO,
               const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
               const BwdParams p) {
  using C = DkvCfg<D>;
  constexpr int NB = C::NB, NSQ = C::NSQ, NSO = C::NSO;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~uintptr_t(1023));
  uint8_t* sK = smem + C::kK;
  uint8_t* sV = smem + C::kV;
  uint8_t* sQ = smem + C::kQ;
  uint8_t* sdO = smem + C::kdO;
  float2* s_stat = reinterpret_cast<float2*>(smem + C::kStat);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kBar);
  uint64_t* bar_kv = bars;              //        K, V landed
  uint64_t* bar_acc = bars + 1;         //        every MMA complete
  uint64_t* bar_st = bars + 2;          //        S^T of an iteration complete
  uint64_t* bar_sl = bars + 3;          //        S^T loaded into registers (8 warps)
  uint64_t* bar_pds = bars + 4;         //        P^T and dS^T written (8 warps)
  uint64_t* bar_sf = bars + 5;          //        row statistics of an iteration written (2 warps)
  uint64_t* bar_dpt = bars + 6;         //        dP^T of an iteration complete
  uint64_t* bar_qf = bars + 7;          // [NSQ]  Q landed
  uint64_t* bar_qe = bar_qf + NSQ;      // [NSQ]  Q stage free (its dK MMAs are complete)
  uint64_t* bar_of = bar_qe + NSQ;      // [NSO]  dO landed
  uint64_t* bar_oe = bar_of + NSO;      // [NSO]  dO stage free (its dV MMAs are complete)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 7 + 2 * NSQ + 2 * NSO);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // grid (kv heads [x parts] x batch, key tiles): key tiles with the most query tiles first
  // (side tile 0 is kept by every later query; the last window tile by the fewest)
  const int kt = SIDE ? int(blockIdx.y) : int(gridDim.y) - 1 - int(blockIdx.y);
  const int G = p.Hq / p.Hkv;
  // the side pass may give each query head of the group its own CTA (and partial buffer)
  const int split = SIDE ? p.split : 1;
  const int n_x = p.Hkv * split;
  const int b = int(blockIdx.x) / n_x;
  const int hk = (int(blockIdx.x) % n_x) / split, part = int(blockIdx.x) % split;
  const int g_lo = (split > 1) ? part : 0, n_g = (split > 1) ? 1 : G;
  const int kv_plane = b * p.Hkv + hk;
  const int ns = min(p.n_side[b], p.side_cap);

  // query tiles [t_lo, t_hi] that keep at least one key of this tile; tiles of padding behind
  // the sequence's last token (seq_len from the index) are left out
  // With document bounds (a packed index) a key is kept by the queries of its own document only:
  // q_end_first / q_end_last are the ends of the documents of the tile's first and last key.
  const DocView dv = doc_view(p.index_header, p.cnt, p.doc_start, p.doc_end);
  const int len = p.seq_len[b];
  const int t_last = (len + kBM - 1) / kBM - 1;
  int t_lo, t_hi, q_end_first = kFar;
  if (SIDE) {
    if (kt * kBN >= ns) return;  // no entries in this side tile: nothing reads its partial rows
    const int32_t* sp = p.side_pos + size_t(b) * p.side_cap;
    t_lo = (sp[kt * kBN] + p.n_neighbor) / kBM;
    t_hi = t_last;
    if (dv.doc_end) {
      q_end_first = dv.doc_end[size_t(b) * p.L + sp[kt * kBN]];
      t_hi = min(t_last, (dv.doc_end[size_t(b) * p.L + sp[min(ns, kt * kBN + kBN) - 1]] - 1) / kBM);
    }
  } else {
    t_lo = kt;  // kBM == kBN
    t_hi = min(t_last, (kt * kBN + kBN - 1 + p.n_neighbor - 1) / kBM);
    if (dv.doc_end && kt * kBN < len) {
      q_end_first = dv.doc_end[size_t(b) * p.L + kt * kBN];
      t_hi = min(t_hi, (dv.doc_end[size_t(b) * p.L + min(len, kt * kBN + kBN) - 1] - 1) / kBM);
    }
  }
  const int n_it = max(0, t_hi - t_lo + 1) * n_g;

  if (tid == 0) {
    mbar_init(bar_kv, 1);
    mbar_init(bar_acc, 1);
    mbar_init(bar_st, 1);
    mbar_init(bar_dpt, 1);
    mbar_init(bar_sl, 8);
    mbar_init(bar_pds, 8);
    mbar_init(bar_sf, 2);
    for (int i = 0; i < NSQ; ++i) { mbar_init(bar_qf + i, 1); mbar_init(bar_qe + i, 1); }
    for (int i = 0; i < NSO; ++i) { mbar_init(bar_of + i, 1); mbar_init(bar_oe + i, 1); }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  bool ok = true;
  auto wait = [&](uint64_t* bar, uint32_t parity) {
    if (!mbar_wait(bar, parity, abort_flag)) {
      if (ok) set_status(p.status, SEPLLM_TIMEOUT);
      ok = false;
    }
  };
  auto q_plane_of = [&](int it) { return b * p.Hq + hk * G + g_lo + it % n_g; };
  // The side pass walks its query tiles from the end of the sequence backwards: the CTAs of
  // neighbouring side tiles of one head, which start together, then read the same Q / dO tiles
  // at the same time (one of them from DRAM, the others from L2) instead of each streaming the
  // head's Q and dO at its own offset.
  auto q0_of = [&](int it) { return (SIDE ? (t_hi - it / n_g) : (t_lo + it / n_g)) * kBM; };

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 104;");
    if (warp == 0 && lane == 0 && n_it > 0) {
      // ---------------- TMA producer ----------------
      mbar_expect_tx(bar_kv, 2 * C::kTile);
      for (int nb = 0; nb < NB; ++nb) {
        tma_load_3d(sK + nb * kTileBlockBytes, &mapK, bar_kv, nb * 64, kt * kBN, kv_plane);
        tma_load_3d(sV + nb * kTileBlockBytes, &mapV, bar_kv, nb * 64, kt * kBN, kv_plane);
      }
      for (int it = 0; it < n_it; ++it) {
        const int sq = it % NSQ, so = it % NSO;
        const int y = q0_of(it), plane = q_plane_of(it);
        if (it >= NSQ) wait(bar_qe + sq, (it / NSQ - 1) & 1);
        mbar_expect_tx(bar_qf + sq, C::kTile);
        for (int nb = 0; nb < NB; ++nb)
          tma_load_3d(sQ + sq * C::kTile + nb * kTileBlockBytes, &mapQ, bar_qf + sq, nb * 64, y, plane);
        if (it >= NSO) wait(bar_oe + so, (it / NSO - 1) & 1);
        mbar_expect_tx(bar_of + so, C::kTile);
        for (int nb = 0; nb < NB; ++nb)
          tma_load_3d(sdO + so * C::kTile + nb * kTileBlockBytes, &mapdO, bar_of + so, nb * 64, y, plane);
      }
    } else if (warp == 1 && lane == 0 && n_it > 0) {
      // ---------------- MMA issuer ----------------
      constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);
      constexpr uint32_t idesc_acc = make_idesc_bf16(128, D, 0, 1);
      const uint32_t k_lo = desc_lo(smem_u32(sK), 16), v_lo = desc_lo(smem_u32(sV), 16);
      const uint32_t q_lo0 = desc_lo(smem_u32(sQ), 16), do_lo0 = desc_lo(smem_u32(sdO), 16);  // K-major B
      const uint32_t qt_lo0 = desc_lo(smem_u32(sQ), kTileBlockBytes);                         // MN-major B
      const uint32_t dot_lo0 = desc_lo(smem_u32(sdO), kTileBlockBytes);
      // ring positions and parities are carried along, not divided out of the iteration counter
      // (the issuing thread's scalar instructions between MMA groups are tensor-pipe idle time)
      auto issue_st = [&](int sq) {
        const uint32_t q_lo = q_lo0 + sq * (C::kTile >> 4);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          umma_ss_lo(tmem + C::kST, k_lo + kmajor_step(k, kTileBlockBytes),
                     q_lo + kmajor_step(k, kTileBlockBytes), idesc_s, k > 0);
        tc_commit(bar_st);
      };
      auto issue_dpt = [&](int so, uint32_t opar) {
        wait(bar_of + so, opar);
        tc_fence_after();
        const uint32_t do_lo = do_lo0 + so * (C::kTile >> 4);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          umma_ss_lo(tmem + C::kdPT, v_lo + kmajor_step(k, kTileBlockBytes),
                     do_lo + kmajor_step(k, kTileBlockBytes), idesc_s, k > 0);
        tc_commit(bar_dpt);
      };
      static_assert(NSO == 2, "the dO ring position is the iteration's parity");
      wait(bar_kv, 0);
      wait(bar_qf, 0);
      tc_fence_after();
      issue_st(0);
      issue_dpt(0, 0);
      int sq = 0;          // Q ring stage of iteration `it`
      uint32_t qpar = 0;   // parity of that stage's "full" barrier
      for (int it = 0; it < n_it; ++it) {
        const uint32_t ipar = uint32_t(it) & 1u;
        int sq1 = sq + 1;
        uint32_t qpar1 = qpar;
        if (sq1 == NSQ) { sq1 = 0; qpar1 ^= 1u; }
        const int so = int(ipar);                       // dO ring stage of iteration `it`
        const uint32_t opar1 = (uint32_t(it + 1) >> 1) & 1u;  // "full" parity of iteration it+1's dO stage
        if (it + 1 < n_it) {
          wait(bar_qf + sq1, qpar1);
          wait(bar_sl, ipar);
          tc_fence_after();
          issue_st(sq1);
        }
        // the next dO tile is waited for here, off the chain that starts with P^T / dS^T below
        if (it + 1 < n_it) wait(bar_of + (so ^ 1), opar1);
        wait(bar_pds, ipar);
        tc_fence_after();
        // Within the dP^T range, warpgroup u's columns [64u, 64u+64) hold P^T of its 64 queries
        // in the first 32 and dS^T in the last 32.  The three groups go to the pipe back to back:
        // every gap in which the pipe runs dry costs a few hundred cycles of start-up on the
        // chain dS^T(it) -> dV, dK, dP^T(it+1) -> dS^T(it+1), so the commits come after them.
        const uint32_t dot_lo = dot_lo0 + so * (C::kTile >> 4);
        const uint32_t qt_lo = qt_lo0 + sq * (C::kTile >> 4);
#pragma unroll
        for (int k = 0; k < kBM / 16; ++k)
          umma_ts_lo(tmem + C::kdV, tmem + C::kdPT + (k >> 2) * 64 + (k & 3) * 8,
                     dot_lo + mnmajor_step(k), idesc_acc, (it > 0 || k > 0));
#pragma unroll
        for (int k = 0; k < kBM / 16; ++k)
          umma_ts_lo(tmem + C::kdK, tmem + C::kdPT + (k >> 2) * 64 + 32 + (k & 3) * 8,
                     qt_lo + mnmajor_step(k), idesc_acc, (it > 0 || k > 0));
        if (it + 1 < n_it) {
          const uint32_t do_lo = do_lo0 + (so ^ 1) * (C::kTile >> 4);
#pragma unroll
          for (int k = 0; k < D / 16; ++k)
            umma_ss_lo(tmem + C::kdPT, v_lo + kmajor_step(k, kTileBlockBytes),
                       do_lo + kmajor_step(k, kTileBlockBytes), idesc_s, k > 0);
          tc_commit(bar_dpt);
        }
        tc_commit(bar_oe + so);
        tc_commit(bar_qe + sq);
        sq = sq1;
        qpar = qpar1;
      }
      tc_commit(bar_acc);
    } else if (warp >= 2) {
      // ---------------- row statistics ----------------
      // one buffer: iteration it's pairs are written once iteration it-1's arithmetic is done
      const int i = tid - 64;  // 0..63
      for (int it = 0; it < n_it; ++it) {
        const int q = q0_of(it) + i;
        const size_t base = size_t(q_plane_of(it)) * p.L;
        const float2 v0 = (q < p.L) ? p.stats[base + q] : make_float2(INFINITY, 0.f);
        const float2 v1 = (q + 64 < p.L) ? p.stats[base + q + 64] : make_float2(INFINITY, 0.f);
        if (it >= 1) wait(bar_pds, (it - 1) & 1);
        // -LSE of the 128 query columns, then -Delta of the 128: the arithmetic warps read two
        // neighbouring columns' values as one packed fp32 pair
        float* sf = reinterpret_cast<float*>(s_stat);
        sf[i] = -v0.x;
        sf[64 + i] = -v1.x;
        sf[128 + i] = -v0.y;
        sf[192 + i] = -v1.y;
        mbar_arrive_warp(bar_sf);
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 200;");
    // ---------------- P^T and dS^T ----------------
    const int u = (warp >= 8) ? 1 : 0;
    const int r = tid & 127;
    const int key = kt * kBN + r;  // side entry index (SIDE) or key position (window)
    const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
    const uint32_t tST = tmem + lane_base + C::kST + u * 64;
    const uint32_t tdPT = tmem + lane_base + C::kdPT + u * 64;
    // queries that keep this key: [q_first, q_end)
    int q_first, q_end, tile_q_max;
    if (SIDE) {
      const int pos = (key < ns) ? p.side_pos[size_t(b) * p.side_cap + key] : -1;
      q_first = (pos >= 0) ? pos + p.n_neighbor : kFar;
      q_end = (pos >= 0 && dv.doc_end) ? dv.doc_end[size_t(b) * p.L + pos] : kFar;
      // first query that keeps every key of the tile (never, if the tile has padding rows)
      tile_q_max = (kt * kBN + kBN <= ns)
                       ? p.side_pos[size_t(b) * p.side_cap + kt * kBN + kBN - 1] + p.n_neighbor
                       : kFar;
    } else {
      q_first = key;
      q_end = key + p.n_neighbor;
      if (dv.doc_end && key < p.L) q_end = min(q_end, dv.doc_end[size_t(b) * p.L + key]);
      tile_q_max = 0;
    }
    for (int it = 0; it < n_it; ++it) {
      const int q0 = q0_of(it);
      const int c_lo = q_first - q0, c_hi = q_end - q0;
      bool need_mask;
      if (SIDE) need_mask = tile_q_max > q0;
      else need_mask = !(kt * kBN + kBN - 1 <= q0 && q0 + kBM - 1 <= kt * kBN + p.n_neighbor - 1);
      need_mask = need_mask || (q0 + kBM > q_end_first);   // a document of the tile ends inside these queries
      // phase A (needs S^T only; runs under the previous iteration's dV / dK and this iteration's
      // dP^T MMAs): P^T = exp2(S^T * scale - LSE), kept in registers
      wait(bar_sf, it & 1);
      wait(bar_st, it & 1);
      tc_fence_after();
      uint32_t sv[2][32];
      tmem_ld32(tST, sv[0]);
      tmem_ld32(tST + 32, sv[1]);
      tmem_ld_wait();
      tc_fence_before();
      mbar_arrive_warp(bar_sl);  // the S^T columns may be overwritten from here on
      // two columns' -LSE (log2 units) and -Delta per shared-memory load, as packed fp32 pairs
      const unsigned long long* nlse2 =
          reinterpret_cast<const unsigned long long*>(reinterpret_cast<const float*>(s_stat) + u * 64);
      const unsigned long long* ndel2 = nlse2 + 64;
      const unsigned long long scale2 = pack_f32x2(p.scale_log2, p.scale_log2);
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          const float2 a = unpack_f32x2(fma_f32x2(
              pack_f32x2(__uint_as_float(sv[c][e]), __uint_as_float(sv[c][e + 1])), scale2,
              nlse2[(c * 32 + e) >> 1]));
          sv[c][e] = __float_as_uint(ex2(a.x));
          sv[c][e + 1] = __float_as_uint(ex2(a.y));
        }
      if (need_mask) {
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const int col = u * 64 + c * 32 + e;
            sv[c][e] = (col >= c_lo && col < c_hi) ? sv[c][e] : 0u;
          }
      }
      // phase B: dS^T = P^T (dP^T - Delta)
      wait(bar_dpt, it & 1);
      tc_fence_after();
      uint32_t pkp[32], pkd[32];
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t dp[32];
        tmem_ld32(tdPT + c * 32, dp);
        tmem_ld_wait();
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          const float p0 = __uint_as_float(sv[c][e]), p1 = __uint_as_float(sv[c][e + 1]);
          pkp[c * 16 + (e >> 1)] = pack_bf16(p0, p1);
          const unsigned long long t2 = add_f32x2(
              pack_f32x2(__uint_as_float(dp[e]), __uint_as_float(dp[e + 1])), ndel2[(c * 32 + e) >> 1]);
          const float2 ds = unpack_f32x2(mul_f32x2(pack_f32x2(p0, p1), t2));
          pkd[c * 16 + (e >> 1)] = pack_bf16(ds.x, ds.y);
        }
      }
      tmem_st32(tdPT, pkp);
      tmem_st32(tdPT + 32, pkd);
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive_warp(bar_pds);
    }

    // ---------------- epilogue: warps 4-7 take dV, warps 8-11 take dK ----------------
    if (n_it > 0) {
      wait(bar_acc, 0);
      tc_fence_after();
    }
    const uint32_t t_acc = tmem + lane_base + (u ? C::kdK : C::kdV);
    const float mul = u ? p.scale : 1.f;
    if (SIDE) {
      // fp32 partial rows for the entries of this side tile
      const bool r_ok = key < p.cap_pad;
      float* base = (u ? p.dKs : p.dVs) +
                    ((size_t(part) * p.B + b) * p.Hkv + hk) * size_t(p.cap_pad) * D +
                    size_t(key) * D;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t rr[32];
        if (n_it > 0) {
          tmem_ld32(t_acc + c * 32, rr);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) rr[e] = 0;
        }
        if (r_ok) {
          float v[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(rr[e]) * mul;
          store_row_chunk32(base, c * 32, 1, v);
        }
      }
    } else {
      // final rows: window part plus, for initial/separator tokens, the side partials of the token
      const bool r_ok = key < p.L;
      int side_idx = -1;
      if (r_ok) {
        const int32_t* cnt_b = p.cnt + size_t(b) * (p.L + 1);
        const int c0 = cnt_b[key], c1 = cnt_b[key + 1];
        if (c1 > c0 && c0 < ns) side_idx = c0;
      }
      const size_t part_stride = size_t(p.B) * p.Hkv * size_t(p.cap_pad) * D;
      const float* part0 = (u ? p.dKs : p.dVs) +
                           (size_t(b) * p.Hkv + hk) * size_t(p.cap_pad) * D +
                           size_t(max(side_idx, 0)) * D;
      void* out = u ? p.dK : p.dV;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t rr[32];
        if (n_it > 0) {
          tmem_ld32(t_acc + c * 32, rr);
          tmem_ld_wait();
        } else {   // a key tile of padding: its rows of dK and dV are written as 0
#pragma unroll
          for (int e = 0; e < 32; ++e) rr[e] = 0;
        }
        if (r_ok) {
          float v[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(rr[e]) * mul;
          if (side_idx >= 0) {
            for (int sp = 0; sp < p.split; ++sp) {
              const float4* src = reinterpret_cast<const float4*>(part0 + sp * part_stride + c * 32);
#pragma unroll
              for (int q = 0; q < 8; ++q) {
                const float4 a = src[q];
                v[4 * q] += a.x; v[4 * q + 1] += a.y; v[4 * q + 2] += a.z; v[4 * q + 3] += a.w;
              }
            }
          }
          store_row_chunk32(out, (size_t(kv_plane) * p.L + key) * p.d + c * 32, p.grad_fp32, v,
                            p.d - c * 32);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

template <int D>
static sepllm_status launch_bwd(const sepllm_attn_desc* d, const sepllm_index_desc* id,
                                const sepllm_index_header& ih, const void* dO, const void* Q,
                                const void* K, const void* V, const void* O, const float* LSE,
                                const uint8_t* index, void* dQ, void* dK, void* dV, uint8_t* ws,
                                cudaStream_t stream) {
  const AttnLayout lay = attn_layout(d, id);
  __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(ws + lay.off_ks);
  __nv_bfloat16* Vs = reinterpret_cast<__nv_bfloat16*>(ws + lay.off_vs);
  const int32_t* side_pos = reinterpret_cast<const int32_t*>(index + ih.off_side_pos);
  const int32_t* n_side = reinterpret_cast<const int32_t*>(index + ih.off_n_side);
  record_event(d, 0, stream);
  if (!(d->flags & SEPLLM_ATTN_SIDE_READY))
    launch_gather(d, id, lay.cap_pad, K, V, side_pos, n_side, Ks, Vs, reinterpret_cast<int32_t*>(ws), stream);
  record_event(d, 1, stream);

  float2* stats = reinterpret_cast<float2*>(ws + lay.off_delta);
  const size_t rows = size_t(d->B) * d->Hq * d->L;
  {
    constexpr int RPB = 256 / (D / 8);
    bwd_delta<D><<<unsigned((rows + RPB - 1) / RPB), 256, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(dO), static_cast<const __nv_bfloat16*>(O), LSE, stats,
        rows, d->d);
  }
  record_event(d, 2, stream);

  CUtensorMap mq, mdo, mk, mv, mks, mvs;
  sepllm_status st;
  const int64_t L = d->L, nq = int64_t(d->B) * d->Hq, nkv = int64_t(d->B) * d->Hkv;
  const int64_t cp = lay.cap_pad, dr = d->d;  // rows of dr elements; the boxes read zeros from dr to D
  if ((st = make_tile_map(&mq, Q, dr, L, nq, dr, L * dr, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mdo, dO, dr, L, nq, dr, L * dr, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mk, K, dr, L, nkv, dr, L * dr, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mv, V, dr, L, nkv, dr, L * dr, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mks, Ks, D, cp, nkv, D, cp * D, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mvs, Vs, D, cp, nkv, D, cp * D, 128)) != SEPLLM_OK) return st;

  BwdParams p;
  p.cnt = reinterpret_cast<const int32_t*>(index + ih.off_cnt);
  p.lim = reinterpret_cast<const int32_t*>(index + ih.off_lim);
  p.side_pos = side_pos;
  p.n_side = n_side;
  p.tile_meta = reinterpret_cast<const int32_t*>(index + ih.off_tile_meta);
  p.seq_len = reinterpret_cast<const int32_t*>(index + ih.off_seq_len);
  p.index_header = reinterpret_cast<const sepllm_index_header*>(index);
  p.doc_start = reinterpret_cast<const int32_t*>(index + ih.off_doc_start);
  p.doc_end = reinterpret_cast<const int32_t*>(index + ih.off_doc_end);
  p.stats = stats;
  p.dKs = reinterpret_cast<float*>(ws + lay.off_dks);
  p.dVs = reinterpret_cast<float*>(ws + lay.off_dvs);
  p.dQ = dQ;
  p.dK = dK;
  p.dV = dV;
  p.status = reinterpret_cast<int32_t*>(ws);
  p.B = d->B;
  p.L = d->L;
  p.d = d->d;
  p.T = ih.n_tiles;
  p.Hq = d->Hq;
  p.Hkv = d->Hkv;
  p.n_neighbor = id->n_neighbor;
  p.side_cap = id->side_cap;
  p.cap_pad = lay.cap_pad;
  p.grad_fp32 = d->grad_dtype;
  p.split = lay.split;
  const int G = d->Hq / d->Hkv;
  p.pair_heads = (G % 2 == 0) ? 1 : 0;
  p.scale = (d->scale != 0.f) ? d->scale : 1.0f / sqrtf(float(d->d));
  p.scale_log2 = p.scale * kLog2e;

  SEPLLM_CUDA_TRY(cudaFuncSetAttribute(bwd_dq_kernel<D, false>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       int(DqCfg<D>::kRequest)));
  SEPLLM_CUDA_TRY(cudaFuncSetAttribute(bwd_dq_kernel<D, true>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       int(DqCfg<D>::kRequest)));
  SEPLLM_CUDA_TRY(cudaFuncSetAttribute(bwd_dkv_kernel<D, true>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       int(DkvCfg<D>::kRequest)));
  SEPLLM_CUDA_TRY(cudaFuncSetAttribute(bwd_dkv_kernel<D, false>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       int(DkvCfg<D>::kRequest)));
  {
    const int n_items = d->Hq * d->B * ih.n_tiles;
    bwd_dq_kernel<D, false><<<std::min(n_items, sm_count()), kBwdThreads, DqCfg<D>::kRequest, stream>>>(
        mk, mv, mks, mvs, static_cast<const __nv_bfloat16*>(Q), static_cast<const __nv_bfloat16*>(dO),
        p, n_items);
    bwd_dq_kernel<D, true><<<std::min(n_items, sm_count()), kBwdThreads, DqCfg<D>::kRequest, stream>>>(
        mk, mv, mks, mvs, static_cast<const __nv_bfloat16*>(Q), static_cast<const __nv_bfloat16*>(dO),
        p, n_items);
  }
  record_event(d, 3, stream);
  bwd_dkv_kernel<D, true><<<dim3(d->Hkv * lay.split * d->B, lay.cap_pad / kBN), kBwdThreads,
                            DkvCfg<D>::kRequest, stream>>>(mq, mdo, mks, mvs, p);
  record_event(d, 4, stream);
  bwd_dkv_kernel<D, false><<<dim3(d->Hkv * d->B, ih.n_tiles), kBwdThreads, DkvCfg<D>::kRequest,
                             stream>>>(mq, mdo, mk, mv, p);
  record_event(d, 5, stream);
  SEPLLM_CUDA_TRY(cudaGetLastError());
  return SEPLLM_OK;
}

}  // namespace sepllm

using namespace sepllm;

extern "C" sepllm_status sepllm_attn_bwd(const sepllm_attn_desc* desc,
                                         const sepllm_index_desc* idesc, const void* dO,
                                         const void* Q, const void* K, const void* V,
                                         const void* O, const float* LSE, const void* index,
                                         void* dQ, void* dK, void* dV, void* workspace,
                                         void* stream_) {
  sepllm_status st = check_attn(desc, idesc);
  if (st != SEPLLM_OK) return st;
  if (!dO || !Q || !K || !V || !O || !LSE || !index || !dQ || !dK || !dV || !workspace)
    return SEPLLM_INVALID_ARG;
  if (!aligned(dO, 16) || !aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) ||
      !aligned(O, 16) || !aligned(dQ, 16) || !aligned(dK, 16) || !aligned(dV, 16) ||
      !aligned(LSE, 4) || !aligned(index, kAlign) || !aligned(workspace, kAlign))
    return SEPLLM_INVALID_ARG;
  sepllm_index_header ih;
  if ((st = fill_index_header(idesc, &ih)) != SEPLLM_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  // A backward that continues on the forward's workspace keeps the forward's status word: a
  // condition the forward recorded stays readable until the caller looks at it.
  // Otherwise the side gather, the call's first launch, resets it.
  const uint8_t* idx = static_cast<const uint8_t*>(index);
  if (kernel_head_dim(desc->d) == 64)
    return launch_bwd<64>(desc, idesc, ih, dO, Q, K, V, O, LSE, idx, dQ, dK, dV, ws, stream);
  return launch_bwd<128>(desc, idesc, ih, dO, Q, K, V, O, LSE, idx, dQ, dK, dV, ws, stream);
}
