// Forward of separator-masked attention (Eq. 1 under the mask of Eq. 2) for query groups of four
// heads at head size 128: the form the long-context and prefill workloads run.
//
// Two CTAs of a cluster form an MMA pair and work on the four query heads of one kv head at one
// query tile: each CTA owns two heads ("slots" 0 and 1, 128 rows each), and every MMA has 256
// rows, the upper half read from and written to the other CTA.  All four tiles walk the same key
// tiles, so each CTA loads only half of every K tile (64 of its 128 keys) and half of every V
// tile (64 of its 128 columns): the B operand of a pair MMA is split over the two CTAs.  The
// shared memory this saves holds P: the softmax threads write P as bf16 into shared memory
// instead of over S in tensor memory, S is free again as soon as it has been read into registers,
// and the MMA thread issues S of the next key tile at once.  The chain "softmax -> P V -> next S
// -> next softmax" of a slot, which bounds a kernel that keeps P over S, is gone: a slot's softmax
// threads go from one key tile to the next without waiting for the tensor pipe.
//
//   warp 0      TMA producer: Q of both slots, then K and V halves through NST-stage rings
//               (loads of both CTAs are counted on the even CTA's barriers; no multicast)
//   warps 1-2   even CTA: MMA issuers for the pair, one thread per slot
//   warps 1-3   odd CTA: relays.  An arrival on a barrier of the other CTA has to be a release at
//               cluster scope, which costs the arriving warp close to a thousand cycles; so the odd
//               CTA's softmax warps arrive on barriers of their own CTA (cheap), and one thread per
//               kind of event waits there and passes a single arrival on to the even CTA
//   warps 4-7   softmax of slot 0, one thread per query row (= tensor-memory lane)
//   warps 8-11  softmax of slot 1
#include "attn_common.cuh"

namespace sepllm {

namespace {

constexpr int kD = 128;
constexpr int kNB = kD / 64;
constexpr int kNST = 3;                                   // K and V ring depth
constexpr uint32_t kQTile = kNB * kTileBlockBytes;        // 128 rows x 128 columns: 32 KB
constexpr uint32_t kKHalfBlock = 64 * 128;                // 64 keys x 64 columns
constexpr uint32_t kKHalf = kNB * kKHalfBlock;            // 64 keys x 128 columns: 16 KB
constexpr uint32_t kVHalf = kTileBlockBytes;              // 128 keys x 64 columns: 16 KB
constexpr uint32_t kPTile = 2 * kTileBlockBytes;          // 128 rows x 128 keys: 32 KB

struct PairSmem {
  static constexpr uint32_t kQ = 0;                       // 2 slots
  static constexpr uint32_t kP = kQ + 2 * kQTile;         // 2 slots
  static constexpr uint32_t kK = kP + 2 * kPTile;
  static constexpr uint32_t kV = kK + kNST * kKHalf;
  static constexpr uint32_t kBar = kV + kNST * kVHalf;
  static constexpr uint32_t kTotal = kBar + 512;
  static constexpr uint32_t kRequest = kTotal + 1024;
  // tensor-memory columns
  static constexpr uint32_t kS0 = 0, kS1 = 128, kO0 = 256, kO1 = 384;
};
static_assert(PairSmem::kRequest <= 227 * 1024, "shared memory budget");

constexpr int kPairThreads = 384;
constexpr long long kSlotOffsetCycles = 1600;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
attn_fwd_pair_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK64,
                     const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapKs64,
                     const __grid_constant__ CUtensorMap mapVs, const FwdParams p) {
  using C = PairSmem;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~uintptr_t(1023));
  uint8_t* sQ = smem + C::kQ;
  uint8_t* sP = smem + C::kP;
  uint8_t* sK = smem + C::kK;
  uint8_t* sV = smem + C::kV;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kBar);
  // Barriers marked (even) are used in the even CTA only and collect both CTAs' loads; bar_sl and
  // bar_p count the CTA's own four softmax warps and, in the even CTA, one more arrival that the
  // odd CTA's relay passes on; the others are signalled in both CTAs at once by the MMA thread's
  // commits.
  uint64_t* bar_q = bars;                    // [2]   (even) Q of slot x of both CTAs landed
  uint64_t* bar_s = bars + 2;                // [2]   S_x complete
  uint64_t* bar_sl = bars + 4;               // [2]   S_x read into registers
  uint64_t* bar_p = bars + 6;                // [2]   P_x written
  uint64_t* bar_pv = bars + 8;               // [2]   P_x V complete: P_x may be rewritten, O_x is at rest
  uint64_t* bar_o = bars + 10;               //       every MMA complete
  uint64_t* bar_kf = bars + 12;              // [NST] (even) K stage full in both CTAs
  uint64_t* bar_ke = bar_kf + kNST;          // [NST] K stage free
  uint64_t* bar_vf = bar_ke + kNST;          // [NST] (even)
  uint64_t* bar_ve = bar_vf + kNST;          // [NST]
  uint64_t* bar_tok = bars + 12 + 4 * kNST;  // [2]   slot x may run its exponentials
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_tok + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();   // 0 = even CTA, issues the MMAs
  // grid (pairs of query heads x batch, tiles), longest tiles first; the two CTAs of a cluster are
  // neighbours in x and hold heads 4g, 4g+1 and 4g+2, 4g+3 of one group
  const int heads_x = p.Hq / 2;
  const int b = int(blockIdx.x) / heads_x, hx = int(blockIdx.x) % heads_x;
  const int t = p.T - 1 - int(blockIdx.y);
  const int G = p.Hq / p.Hkv;
  if (t * kBM >= p.seq_len[b]) return;   // a tile of padding (the same for both CTAs of the pair)
  const DocView dv = doc_view(p.index_header, p.cnt, p.doc_start, p.doc_end);
  const SlotGeom g = load_slot(p.tile_meta, p.seq_len, b, p.T, t, 2 * hx, p.side_tiles_cap, dv, p.L,
                               p.n_neighbor);
  const int kv_plane = b * p.Hkv + (2 * hx) / G;
  // key tiles: side tiles [sbase, sbase + ns), then window tiles [wlo, whi)
  const int sbase = g.s0, ns = max(0, g.ns - g.s0), wlo = g.wlo;
  const int n_tiles = ns + (g.whi - g.wlo);

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_q + i, 1);
      mbar_init(bar_s + i, 1);
      mbar_init(bar_sl + i, rank == 0 ? 5 : 4);
      mbar_init(bar_p + i, rank == 0 ? 5 : 4);
      mbar_init(bar_pv + i, 1);
      mbar_init(bar_tok + i, 4);
    }
    mbar_init(bar_o, 2);   // one commit from each of the two issuing threads
    for (int i = 0; i < kNST; ++i) {
      mbar_init(bar_kf + i, 1); mbar_init(bar_ke + i, 2); mbar_init(bar_vf + i, 1); mbar_init(bar_ve + i, 2);
    }
    *abort_flag = 0;
    fence_mbar_init();
    tma_prefetch_desc(&mapQ); tma_prefetch_desc(&mapK64); tma_prefetch_desc(&mapV);
    tma_prefetch_desc(&mapKs64); tma_prefetch_desc(&mapVs);
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc_pair(tmem_slot, 512);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // both CTAs' barriers and tensor memory exist before anyone signals across
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  bool ok = true;
  auto wait = [&](uint64_t* bar, uint32_t parity) {
    if (!mbar_wait(bar, parity, abort_flag)) {
      if (ok) set_status(p.status, SEPLLM_TIMEOUT);
      ok = false;
    }
  };
  // a barrier the other CTA's relay arrives on
  auto wait_cluster = [&](uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait_cluster(bar, parity)) return;
    const long long t0 = clock64();
    while (!mbar_try_wait_cluster(bar, parity)) {
      if (*abort_flag || clock64() - t0 > kWaitCycles) {
        *abort_flag = 1;
        if (ok) set_status(p.status, SEPLLM_TIMEOUT);
        ok = false;
        return;
      }
    }
  };
  // the even CTA's copy of a barrier, as a cluster-wide address
  auto even = [&](uint64_t* bar) { return map_to_cta(smem_u32(bar), 0); };

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (warp == 0 && lane == 0) {
      // ---------------- TMA producer (both CTAs) ----------------
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        if (rank == 0) mbar_expect_tx(bar_q + x, 2 * kQTile);
        const uint32_t bq = even(bar_q + x);
        for (int nb = 0; nb < kNB; ++nb)
          tma_load_3d_pair(sQ + x * kQTile + nb * kTileBlockBytes, &mapQ, bq, nb * 64, t * kBM,
                           b * p.Hq + 2 * hx + x);
      }
      for (int j = 0; j < n_tiles; ++j) {
        const int st = j % kNST, use = j / kNST;
        const bool side = j < ns;
        const int y = side ? (sbase + j) * kBN : (wlo + (j - ns)) * kBN;
        // K: this CTA's 64 keys of the tile, all 128 columns
        if (use > 0) wait(bar_ke + st, (use - 1) & 1);
        if (rank == 0) mbar_expect_tx(bar_kf + st, 2 * kKHalf);
        const uint32_t bk = even(bar_kf + st);
        for (int nb = 0; nb < kNB; ++nb)
          tma_load_3d_pair(sK + st * kKHalf + nb * kKHalfBlock, side ? &mapKs64 : &mapK64, bk, nb * 64,
                           y + 64 * int(rank), kv_plane);
        // V: all 128 keys of the tile, this CTA's 64 columns
        if (use > 0) wait(bar_ve + st, (use - 1) & 1);
        if (rank == 0) mbar_expect_tx(bar_vf + st, 2 * kVHalf);
        tma_load_3d_pair(sV + st * kVHalf, side ? &mapVs : &mapV, even(bar_vf + st), 64 * int(rank), y,
                         kv_plane);
      }
    } else if ((warp == 1 || warp == 2) && lane == 0 && rank == 0) {
      // ---------------- MMA issuers (even CTA): warp 1 for slot 0, warp 2 for slot 1 ----------------
      // Between two groups of eight MMAs the issuing thread spends a few hundred cycles on waits,
      // a fence and a commit, and the tensor pipe holds next to no queue; with one thread per slot
      // one thread's MMAs run while the other is between groups.  A slot's groups go in its own
      // order: S(j+1) as soon as S(j) has been read, P V(j) as soon as P(j) is written.
      const int x = warp - 1;
      constexpr uint32_t idesc_s = make_idesc_bf16(256, 128, 0, 0);
      constexpr uint32_t idesc_o = make_idesc_bf16(256, kD, 0, 1);
      const uint32_t q_lo = desc_lo(smem_u32(sQ + x * kQTile), 16);
      const uint32_t p_lo = desc_lo(smem_u32(sP + x * kPTile), 16);
      const uint32_t k_lo0 = desc_lo(smem_u32(sK), 16);
      const uint32_t v_lo0 = desc_lo(smem_u32(sV), kTileBlockBytes);
      const uint32_t tS = tmem + (x ? C::kS1 : C::kS0), tO = tmem + (x ? C::kO1 : C::kO0);
      auto issue_s = [&](int j) {
        const int st = j % kNST;
        wait(bar_kf + st, (j / kNST) & 1);
        tc_fence_after();
        const uint32_t k_lo = k_lo0 + st * (kKHalf >> 4);
#pragma unroll
        for (int k = 0; k < kD / 16; ++k)
          umma_ss_lo_pair(tS, q_lo + kmajor_step(k, kTileBlockBytes), k_lo + kmajor_step(k, kKHalfBlock),
                          idesc_s, k > 0);
        tc_commit_pair(bar_s + x, 3);
        tc_commit_pair(bar_ke + st, 3);   // one of the two arrivals that free the stage
      };
      wait(bar_q + x, 0);
      if (x == 1) {
        // Slot 1 starts half a softmax period after slot 0.  The two slots' softmax warps share
        // the exponential unit; in step they would both sit in their exponentials at once (twice as
        // long) and then both in their loads and stores; out of step one slot's exponentials run
        // under the other's loads and stores.  Nothing couples the slots afterwards, so the offset
        // stays.
        const long long t0 = clock64();
        while (clock64() - t0 < kSlotOffsetCycles) {}
      }
      issue_s(0);
      for (int j = 0; j < n_tiles; ++j) {
        if (j + 1 < n_tiles) {
          wait_cluster(bar_sl + x, j & 1);
          issue_s(j + 1);
        }
        const int st = j % kNST;
        wait_cluster(bar_p + x, j & 1);
        wait(bar_vf + st, (j / kNST) & 1);
        tc_fence_after();
        const uint32_t v_lo = v_lo0 + st * (kVHalf >> 4);
#pragma unroll
        for (int k = 0; k < kBN / 16; ++k)
          umma_ss_lo_pair(tO, p_lo + kmajor_step(k, kTileBlockBytes), v_lo + mnmajor_step(k), idesc_o,
                          (j > 0 || k > 0));
        tc_commit_pair(bar_pv + x, 3);
        tc_commit_pair(bar_ve + st, 3);
      }
      tc_commit_pair(bar_o, 3);
    } else if (rank == 1 && warp >= 1 && lane == 0) {
      // ---------------- relays (odd CTA) ----------------
      if (warp <= 2) {
        // "S_x read" of slot x = warp - 1
        const int x = warp - 1;
        const uint32_t dst = even(bar_sl + x);
        for (int j = 0; j + 1 < n_tiles; ++j) {   // the last tile's is needed by no one
          wait(bar_sl + x, j & 1);
          mbar_arrive_cluster(dst);
        }
      } else {
        // "P_x written" of both slots, whichever comes first
        const uint32_t dst[2] = {even(bar_p), even(bar_p + 1)};
        int jr[2] = {0, 0};
        long long t_last = clock64();
        while (jr[0] < n_tiles || jr[1] < n_tiles) {
          bool progressed = false;
#pragma unroll
          for (int x = 0; x < 2; ++x)
            if (jr[x] < n_tiles && mbar_try_wait(bar_p + x, jr[x] & 1)) {
              mbar_arrive_cluster(dst[x]);
              ++jr[x];
              progressed = true;
            }
          if (progressed) {
            t_last = clock64();
          } else if (*abort_flag || clock64() - t_last > kWaitCycles) {
            *abort_flag = 1;
            if (ok) set_status(p.status, SEPLLM_TIMEOUT);
            ok = false;
            break;
          }
        }
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    // ---------------- softmax of slot x (both CTAs) ----------------
    const int x = (warp >= 8) ? 1 : 0;
    const int r = tid & 127;                       // row in the tile = tensor-memory lane
    const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_base + (x ? C::kS1 : C::kS0);
    const uint32_t tO = tmem + lane_base + (x ? C::kO1 : C::kO0);
    uint8_t* sPx = sP + x * kPTile;
    const int hq = 2 * hx + x;
    const int row = t * kBM + r;  // this thread's query position
    const int q_plane = b * p.Hq + hq;
    const RowGeom rg = row_geom(p.lim, dv, b, p.L, row, p.n_neighbor, p.side_cap);
    float m_ref = -INFINITY;  // reference exponent (log2 units), may lag the true row maximum
    float l_sum = 0.f;
    uint32_t sreg[4][32];
    for (int j = 0; j < n_tiles; ++j) {
      wait(bar_s + x, j & 1);
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, sreg[c]);
      tmem_ld_wait();
      tc_fence_before();
      mbar_arrive_warp(bar_sl + x);   // S_x may be overwritten by the next key tile's scores

      // kept columns of this tile for this row: [c_lo, c_hi)
      const bool side = j < ns;
      int c_lo, c_hi;
      bool need_mask;
      key_range(side, side ? sbase + j : wlo + (j - ns), g, row, rg, c_lo, c_hi, need_mask);
      if (need_mask) {
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const int col = c * 32 + e;
            sreg[c][e] = (col >= c_lo && col < c_hi) ? sreg[c][e] : 0xff800000u;  // -inf
          }
      }
      // The reference exponent moves only when the tile's maximum exceeds it by more than 2^8
      // (fp32 sums and bf16 P have the range for that lag), so O is rarely rescaled.
      float mx;
      {
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int e = 0; e < 32; e += 8)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              mx4[k] = max3(mx4[k], __uint_as_float(sreg[c][e + k]), __uint_as_float(sreg[c][e + 4 + k]));
        mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
      }
      float corr = 1.f;
      bool rescale = false;
      if (mx > m_ref + 8.f) {
        corr = (m_ref == -INFINITY) ? 0.f : ex2(m_ref - mx);
        m_ref = mx;
        rescale = true;
      }
      // P = 2^(S * scale - m_ref), packed as bf16 pairs over sreg[c][0..15].  The two slots take
      // turns at this block: side by side they halve each other's rate at the special-function
      // unit, in turn one slot's exponentials run under the other slot's loads, maxima and stores.
      float tile_sum;
      if (x == 1 || j > 0) wait(bar_tok + x, (x == 1) ? (j & 1) : ((j - 1) & 1));
      {
        const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
        const unsigned long long scale2 = pack_f32x2(p.scale_log2, p.scale_log2);
        const unsigned long long negm2 = pack_f32x2(neg_m, neg_m);
        unsigned long long ps2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float2 a = unpack_f32x2(fma_f32x2(
                pack_f32x2(__uint_as_float(sreg[c][e]), __uint_as_float(sreg[c][e + 1])), scale2, negm2));
            const float p0 = ex2(a.x), p1 = ex2(a.y);
            ps2[(e >> 1) & 3] = add_f32x2(ps2[(e >> 1) & 3], pack_f32x2(p0, p1));
            sreg[c][e >> 1] = pack_bf16(p0, p1);
          }
        const float2 sm = unpack_f32x2(add_f32x2(add_f32x2(ps2[0], ps2[1]), add_f32x2(ps2[2], ps2[3])));
        tile_sum = sm.x + sm.y;
      }
      if (x == 0 || j + 1 < n_tiles) mbar_arrive_warp(bar_tok + (x ^ 1));
      l_sum = l_sum * corr + tile_sum;

      // P_x of the previous key tile has been consumed: the buffer is free and O_x is at rest
      if (j > 0) {
        wait(bar_pv + x, (j - 1) & 1);
        tc_fence_after();
        if (__any_sync(0xffffffffu, rescale)) {
          uint32_t oreg[32];
#pragma unroll
          for (int c = 0; c < kD / 32; ++c) {
            tmem_ld32(tO + c * 32, oreg);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) oreg[e] = __float_as_uint(__uint_as_float(oreg[e]) * corr);
            tmem_st32(tO + c * 32, oreg);
          }
          tmem_st_wait();
          tc_fence_before();
        }
      }
      // P row r: 16 chunks of 8 keys, chunk q of the row at block q / 8, swizzled position q % 8
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int q = 4 * c + i;
          *reinterpret_cast<uint4*>(sPx + (q >> 3) * kTileBlockBytes + swz128(uint32_t(r), uint32_t(q & 7))) =
              make_uint4(sreg[c][4 * i], sreg[c][4 * i + 1], sreg[c][4 * i + 2], sreg[c][4 * i + 3]);
        }
      fence_proxy_async_smem();
      mbar_arrive_warp(bar_p + x);
    }

    wait(bar_o, 0);
    tc_fence_after();
    const float inv_l = (l_sum > 0.f) ? 1.f / l_sum : 0.f;
    if (row < p.L) p.LSE[size_t(q_plane) * p.L + row] = (m_ref + log2f(l_sum)) * 0.6931471805599453f;
    __nv_bfloat16* orow = p.O + (size_t(q_plane) * p.L + row) * p.d;
#pragma unroll
    for (int c = 0; c < kD / 32; ++c) {
      uint32_t oreg[32];
      tmem_ld32(tO + c * 32, oreg);
      tmem_ld_wait();
      if (row < p.L) {
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint4 val;
          val.x = pack_bf16(__uint_as_float(oreg[q4 * 8 + 0]) * inv_l, __uint_as_float(oreg[q4 * 8 + 1]) * inv_l);
          val.y = pack_bf16(__uint_as_float(oreg[q4 * 8 + 2]) * inv_l, __uint_as_float(oreg[q4 * 8 + 3]) * inv_l);
          val.z = pack_bf16(__uint_as_float(oreg[q4 * 8 + 4]) * inv_l, __uint_as_float(oreg[q4 * 8 + 5]) * inv_l);
          val.w = pack_bf16(__uint_as_float(oreg[q4 * 8 + 6]) * inv_l, __uint_as_float(oreg[q4 * 8 + 7]) * inv_l);
          if (c * 32 + q4 * 8 < p.d) *reinterpret_cast<uint4*>(orow + c * 32 + q4 * 8) = val;
        }
      }
    }
  }
  // Neither CTA leaves (or frees tensor memory the pair's MMAs write) before both are done.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 0) tmem_dealloc_pair(tmem, 512);
}

}  // namespace

sepllm_status launch_fwd_pair(const sepllm_attn_desc* d, const FwdParams& p, int n_tiles,
                              const CUtensorMap& mq, const CUtensorMap& mk64, const CUtensorMap& mv,
                              const CUtensorMap& mks64, const CUtensorMap& mvs, cudaStream_t stream) {
  const uint32_t smem = PairSmem::kRequest;
  SEPLLM_CUDA_TRY(cudaFuncSetAttribute(attn_fwd_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       int(smem)));
  // x = pairs of query heads of every sequence: even, and a cluster never straddles two kv heads
  const dim3 grid(d->Hq / 2 * d->B, n_tiles);
  attn_fwd_pair_kernel<<<grid, kPairThreads, smem, stream>>>(mq, mk64, mv, mks64, mvs, p);
  SEPLLM_CUDA_TRY(cudaGetLastError());
  return SEPLLM_OK;
}

}  // namespace sepllm
