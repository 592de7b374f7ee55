// Forward of separator-masked attention (Eq. 1 under the mask of Eq. 2) for sm_100a.
//
// Per query tile of 128 rows the kept keys fall in two groups that never overlap:
//   side   entries [0, lim[i]) of the per-sequence side buffer (initial tokens and separators at
//          distance >= n from the row), gathered once into contiguous K/V side buffers;
//   window keys i-n < j <= i, read from K/V in place.
// A CTA walks the side tiles and then the window tiles of its query tiles: TMA brings 128-key
// K/V tiles into shared memory, tcgen05 MMAs compute S = Q K^T into tensor memory, one thread
// per query row (= tensor-memory lane) runs the online softmax, P returns to tensor memory as
// bf16 and a second MMA accumulates O += P V there.  Only tiles crossing lim[], the diagonal or
// the window's left edge are masked element by element.
#include "attn_common.cuh"

namespace sepllm {

// ---------------------------------------------------------------------------
// host: tensor maps
// ---------------------------------------------------------------------------
EncodeTiledFn get_encode_tiled() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) !=
          cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

sepllm_status make_tile_map(CUtensorMap* map, const void* base, int d, int64_t rows,
                            int64_t planes, int64_t row_stride_elems, int64_t plane_stride_elems,
                            int box_rows) {
  EncodeTiledFn enc = get_encode_tiled();
  if (!enc) return SEPLLM_CUDA_ERROR;
  if (!aligned(base, 16) || (row_stride_elems * 2) % 16 != 0 || (plane_stride_elems * 2) % 16 != 0)
    return SEPLLM_INVALID_ARG;
  cuuint64_t dims[3] = {cuuint64_t(d), cuuint64_t(rows), cuuint64_t(planes)};
  cuuint64_t strides[2] = {cuuint64_t(row_stride_elems) * 2, cuuint64_t(plane_stride_elems) * 2};
  cuuint32_t box[3] = {64, cuuint32_t(box_rows), 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims,
                   strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SEPLLM_OK : SEPLLM_CUDA_ERROR;
}

// ---------------------------------------------------------------------------
// side K/V gather
// ---------------------------------------------------------------------------
// grid (ceil(cap_pad / rows_per_block), Hkv, B).  Row r of the side buffer is K/V row
// side_pos[r]; rows from n_side up to the next multiple of 128 are zero so that the tile holding
// the last entries contains only finite numbers.  Source rows have d elements, side rows D >= d
// (columns from d on are zero).
template <int D>
__global__ void __launch_bounds__(256)
gather_side_kv(const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V,
               const int32_t* __restrict__ side_pos, const int32_t* __restrict__ n_side, int L,
               int d, int Hkv, int side_cap, int cap_pad, __nv_bfloat16* __restrict__ Ks,
               __nv_bfloat16* __restrict__ Vs, int32_t* __restrict__ status) {
  constexpr int LPR = D / 8;
  constexpr int RPB = 256 / LPR;
  const int b = blockIdx.z, hk = blockIdx.y;
  if (threadIdx.x == 0 && (blockIdx.x | blockIdx.y | blockIdx.z) == 0) *status = SEPLLM_OK;
  const int r = blockIdx.x * RPB + threadIdx.x / LPR, l = threadIdx.x % LPR;
  const int ns = min(n_side[b], side_cap);
  const int ns_pad = min(cap_pad, (ns + 127) / 128 * 128);
  if (r >= ns_pad) return;
  const size_t plane = size_t(b) * Hkv + hk;
  uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
  if (r < ns) {
    const int pos = side_pos[size_t(b) * side_cap + r];
    if (pos >= 0 && pos < L && l * 8 < d) {
      kv = *reinterpret_cast<const uint4*>(K + (plane * L + pos) * d + l * 8);
      vv = *reinterpret_cast<const uint4*>(V + (plane * L + pos) * d + l * 8);
    }
  }
  *reinterpret_cast<uint4*>(Ks + (plane * cap_pad + r) * D + l * 8) = kv;
  *reinterpret_cast<uint4*>(Vs + (plane * cap_pad + r) * D + l * 8) = vv;
}

// ---------------------------------------------------------------------------
// forward kernel
// ---------------------------------------------------------------------------
// One CTA works on two query tiles ("slots") that share their key tiles: two query heads of one
// GQA group at the same tile position when the group size is even, else two adjacent tiles of
// one head.  Twelve warps:
//   warp 0      TMA producer: Q of both slots, then the K and V tiles through NST-stage rings
//   warp 1      MMA issuer:   S_x = Q_x K^T and O_x += P_x V for both slots, all in tensor memory
//   warps 4-7   softmax of slot 0, one thread per query row (= tensor-memory lane)
//   warps 8-11  softmax of slot 1
// P never touches shared memory: the softmax threads write it as packed bf16 over the first half
// of their slot's S columns and the PV MMA takes its A operand from tensor memory.  The issuer
// alternates slots, so one slot's softmax runs under the other slot's MMAs.
template <int D>
struct FwdCfg {
  static constexpr int NB = D / 64;                 // 64-column blocks per row
  static constexpr int NST = (D == 128) ? 2 : 4;    // K and V ring depth
  static constexpr uint32_t kTile = NB * kTileBlockBytes;
  static constexpr uint32_t kQ = 0;
  static constexpr uint32_t kK = kQ + 2 * kTile;
  static constexpr uint32_t kV = kK + NST * kTile;
  static constexpr uint32_t kBar = kV + NST * kTile;
  static constexpr uint32_t kTotal = kBar + 512;
  static constexpr uint32_t kRequest = kTotal + 1024;  // > half an SM: one CTA per SM owns all 512 TMEM columns
  // tensor-memory columns
  static constexpr uint32_t kS0 = 0, kS1 = 128, kO0 = 256, kO1 = 256 + D;
};

constexpr int kFwdThreads = 384;

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapKs,
                const __grid_constant__ CUtensorMap mapVs, const FwdParams p) {
  using C = FwdCfg<D>;
  constexpr int NB = C::NB, NST = C::NST;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~uintptr_t(1023));
  uint8_t* sQ = smem + C::kQ;
  uint8_t* sK = smem + C::kK;
  uint8_t* sV = smem + C::kV;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kBar);
  uint64_t* bar_q = bars;                   // [2]   Q of slot x landed
  uint64_t* bar_s = bars + 2;               // [2]   S_x complete (and every earlier MMA)
  uint64_t* bar_p = bars + 4;               // [2]   P_x written by the 4 softmax warps of slot x
  uint64_t* bar_o = bars + 6;               //       every MMA of the CTA complete
  uint64_t* bar_kf = bars + 8;              // [NST] K stage full
  uint64_t* bar_ke = bar_kf + NST;          // [NST] K stage free
  uint64_t* bar_vf = bar_ke + NST;          // [NST]
  uint64_t* bar_ve = bar_vf + NST;          // [NST]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8 + 4 * NST);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // grid (heads x batch, tiles): consecutive CTAs take the same tile position of every head and
  // sequence, longest tiles first, so work is handed out longest-first over the whole launch and
  // the heads of a GQA group find their K/V tiles in L2
  const int G = p.Hq / p.Hkv;
  const int heads_x = p.pair_heads ? p.Hq / 2 : p.Hq;
  const int b = int(blockIdx.x) / heads_x, hx = int(blockIdx.x) % heads_x;

  // the two slots of this CTA (a slot is empty when its tile does not exist or holds only padding)
  SlotGeom g0, g1;
  const DocView dv = doc_view(p.index_header, p.cnt, p.doc_start, p.doc_end);
  if (p.pair_heads) {
    const int t = p.T - 1 - int(blockIdx.y);
    g0 = load_slot(p.tile_meta, p.seq_len, b, p.T, t, 2 * hx, p.side_tiles_cap, dv, p.L, p.n_neighbor);
    g1 = load_slot(p.tile_meta, p.seq_len, b, p.T, t, 2 * hx + 1, p.side_tiles_cap, dv, p.L, p.n_neighbor);
  } else {
    const int t = p.T - 1 - 2 * int(blockIdx.y);
    g0 = load_slot(p.tile_meta, p.seq_len, b, p.T, t - 1, hx, p.side_tiles_cap, dv, p.L, p.n_neighbor);
    g1 = load_slot(p.tile_meta, p.seq_len, b, p.T, t, hx, p.side_tiles_cap, dv, p.L, p.n_neighbor);
  }
  if (g0.t < 0 && g1.t < 0) return;   // both tiles are padding: nothing to do, nothing written
  const int kv_plane = b * p.Hkv + g1.hq / G;
  // key tiles of the CTA: side tiles [sbase, sbase + ns), then window tiles [wlo, whi)
  const int sbase = min(g0.s0, g1.s0);
  const int ns = max(0, max(g0.ns, g1.ns) - sbase);
  const int wlo = min(g0.wlo, g1.wlo);
  const int whi = max(g0.whi, g1.whi);
  const int n_tiles = ns + (whi - wlo);

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) { mbar_init(bar_q + i, 1); mbar_init(bar_s + i, 1); mbar_init(bar_p + i, 4); }
    mbar_init(bar_o, 1);
    for (int i = 0; i < NST; ++i) {
      mbar_init(bar_kf + i, 1); mbar_init(bar_ke + i, 1); mbar_init(bar_vf + i, 1); mbar_init(bar_ve + i, 1);
    }
    *abort_flag = 0;
    fence_mbar_init();
    tma_prefetch_desc(&mapQ); tma_prefetch_desc(&mapK); tma_prefetch_desc(&mapV);
    tma_prefetch_desc(&mapKs); tma_prefetch_desc(&mapVs);
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

  // When the two slots are the two heads of one query tile they walk the same key tiles, and a
  // softmax thread of slot 1 can report the K and V stages free (a commit costs the MMA thread
  // about 90 cycles during which the tensor pipe has nothing queued).
  const bool free_by_softmax = p.pair_heads && g0.t >= 0 && g1.t >= 0;
  bool ok = true;
  auto wait = [&](uint64_t* bar, uint32_t parity) {
    if (!mbar_wait(bar, parity, abort_flag)) {
      if (ok) set_status(p.status, SEPLLM_TIMEOUT);
      ok = false;
    }
  };

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (warp == 0 && lane == 0) {
      // ---------------- TMA producer ----------------
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        const SlotGeom& g = x ? g1 : g0;
        if (g.t >= 0) {
          mbar_expect_tx(bar_q + x, C::kTile);
          for (int nb = 0; nb < NB; ++nb)
            tma_load_3d(sQ + x * C::kTile + nb * kTileBlockBytes, &mapQ, bar_q + x, nb * 64,
                        g.t * kBM, b * p.Hq + g.hq);
        }
      }
      for (int j = 0; j < n_tiles; ++j) {
        const int st = j % NST, use = j / NST;
        const bool side = j < ns;
        const int y = side ? (sbase + j) * kBN : (wlo + (j - ns)) * kBN;
        if (use > 0) wait(bar_ke + st, (use - 1) & 1);
        mbar_expect_tx(bar_kf + st, C::kTile);
        for (int nb = 0; nb < NB; ++nb)
          tma_load_3d(sK + st * C::kTile + nb * kTileBlockBytes, side ? &mapKs : &mapK, bar_kf + st,
                      nb * 64, y, kv_plane);
        if (use > 0) wait(bar_ve + st, (use - 1) & 1);
        mbar_expect_tx(bar_vf + st, C::kTile);
        for (int nb = 0; nb < NB; ++nb)
          tma_load_3d(sV + st * C::kTile + nb * kTileBlockBytes, side ? &mapVs : &mapV, bar_vf + st,
                      nb * 64, y, kv_plane);
      }
    } else if (warp == 1 && lane == 0) {
      // ---------------- MMA issuer ----------------
      constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);
      constexpr uint32_t idesc_o = make_idesc_bf16(128, D, 0, 1);
      const uint32_t q_lo[2] = {desc_lo(smem_u32(sQ), 16), desc_lo(smem_u32(sQ + C::kTile), 16)};
      const uint32_t k_lo0 = desc_lo(smem_u32(sK), 16);
      const uint32_t v_lo0 = desc_lo(smem_u32(sV), kTileBlockBytes);
      int n_pv[2] = {0, 0};  // PV MMAs issued per slot
      bool q_seen[2] = {false, false};
      // Every barrier test, fence and commit costs this thread 50-300 cycles during which the
      // tensor pipe drains, so each is done once per step: the K and V tiles are waited for by
      // the first slot that needs them, and the only tcgen05 fence follows the wait for P (the
      // other waits guard TMA data, which the barrier itself makes visible).
      for (int s = 0; s <= n_tiles; ++s) {
        bool k_waited = false, v_waited = false;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          const SlotGeom& g = x ? g1 : g0;
          const uint32_t tS = tmem + (x ? C::kS1 : C::kS0), tO = tmem + (x ? C::kO1 : C::kO0);
          if (s >= 1 && slot_active(g, sbase, ns, wlo, s - 1)) {
            const int j = s - 1, st = j % NST;
            wait(bar_p + x, n_pv[x] & 1);
            if (!v_waited) { wait(bar_vf + st, (j / NST) & 1); v_waited = true; }
            tc_fence_after();
            const uint32_t v_lo = v_lo0 + st * (C::kTile >> 4);
            umma_ts_lo(tO, tS, v_lo, idesc_o, n_pv[x] > 0);
#pragma unroll
            for (int k = 1; k < kBN / 16; ++k)
              umma_ts_lo(tO, tS + k * 8, v_lo + mnmajor_step(k), idesc_o, 1);
            ++n_pv[x];
          }
          if (s < n_tiles && slot_active(g, sbase, ns, wlo, s)) {
            const int st = s % NST;
            if (!q_seen[x]) { wait(bar_q + x, 0); q_seen[x] = true; }
            if (!k_waited) { wait(bar_kf + st, (s / NST) & 1); k_waited = true; }
            const uint32_t k_lo = k_lo0 + st * (C::kTile >> 4);
#pragma unroll
            for (int k = 0; k < D / 16; ++k)
              umma_ss_lo(tS, q_lo[x] + kmajor_step(k, kTileBlockBytes),
                         k_lo + kmajor_step(k, kTileBlockBytes), idesc_s, k > 0);
            tc_commit(bar_s + x);
          }
        }
        if (!free_by_softmax) {
          if (s < n_tiles) tc_commit(bar_ke + s % NST);      // every S MMA reading K(s) is issued
          if (s >= 1) tc_commit(bar_ve + (s - 1) % NST);     // every PV MMA reading V(s-1) is issued
        }
      }
      tc_commit(bar_o);
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    // ---------------- softmax of slot x ----------------
    const int x = (warp >= 8) ? 1 : 0;
    const int r = tid & 127;                       // row in the tile = tensor-memory lane
    const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_base + (x ? C::kS1 : C::kS0);
    const uint32_t tO = tmem + lane_base + (x ? C::kO1 : C::kO0);
    const SlotGeom g = x ? g1 : g0;
    const int t = g.t;
    if (t >= 0) {
      const int row = t * kBM + r;  // this thread's query position
      const int q_plane = b * p.Hq + g.hq;
      const RowGeom rg = row_geom(p.lim, dv, b, p.L, row, p.n_neighbor, p.side_cap);
      float m_ref = -INFINITY;  // reference exponent (log2 units), may lag the true row maximum
      float l_sum = 0.f;
      int n_done = 0;
      uint32_t sreg[4][32];
      for (int j = 0; j < n_tiles; ++j) {
        if (!slot_active(g, sbase, ns, wlo, j)) continue;
        wait(bar_s + x, n_done & 1);
        tc_fence_after();
        // MMAs complete in issue order: S of slot 1 for tile j done means both slots' S MMAs have
        // read K(j) and both PV MMAs have read V(j-1)
        if (free_by_softmax && tid == 256) {
          mbar_arrive(bar_ke + j % NST);
          if (j >= 1) mbar_arrive(bar_ve + (j - 1) % NST);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, sreg[c]);
        tmem_ld_wait();

        // kept columns of this tile for this row: [c_lo, c_hi)
        const bool side = j < ns;
        int c_lo, c_hi;
        bool need_mask;
        key_range(side, side ? sbase + j : wlo + (j - ns), g, row, rg, c_lo, c_hi, need_mask);
        // Reference exponent.  A tile that needs no mask and finds a reference already set skips
        // the maximum: its exponentials are taken against the old reference, which is exact as
        // long as nothing overflows (fp32 sums and bf16 P have the range for a lag of 2^64), and
        // the row sum tells if it did.  Otherwise the reference moves when the tile's maximum
        // exceeds it by more than 2^8.
        auto tile_max = [&]() -> float {
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int e = 0; e < 32; e += 8)
#pragma unroll
              for (int k = 0; k < 4; ++k)
                mx4[k] = max3(mx4[k], __uint_as_float(sreg[c][e + k]), __uint_as_float(sreg[c][e + 4 + k]));
          return fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
        };
        // P = 2^(S * scale - m_ref) packed over sreg[c][0..15]; returns the row sum of the tile
        auto exponentials = [&]() -> float {
          const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
          const unsigned long long scale2 = pack_f32x2(p.scale_log2, p.scale_log2);
          const unsigned long long negm2 = pack_f32x2(neg_m, neg_m);
          unsigned long long ps2[4] = {0ull, 0ull, 0ull, 0ull};  // four packed partial sums
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
          return sm.x + sm.y;
        };
        auto move_reference = [&](float mx, float& corr, bool& rescale) {
          if (mx > m_ref + 8.f) {
            corr = (m_ref == -INFINITY) ? 0.f : ex2(m_ref - mx);
            m_ref = mx;
            rescale = true;
          }
        };
        if (need_mask) {
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const int col = c * 32 + e;
              sreg[c][e] = (col >= c_lo && col < c_hi) ? sreg[c][e] : 0xff800000u;  // -inf
            }
        }
        float corr = 1.f;
        bool rescale = false;
        if (need_mask || m_ref == -INFINITY) move_reference(tile_max(), corr, rescale);
        float tile_sum = exponentials();
        if (__any_sync(0xffffffffu, !(tile_sum < 1.8e19f))) {
          // some row of this warp ran past the range: take the tile again with its own maximum
#pragma unroll
          for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, sreg[c]);
          tmem_ld_wait();
          move_reference(tile_max(), corr, rescale);
          tile_sum = exponentials();
        }
        l_sum = l_sum * corr + tile_sum;

        // S_x(j) complete means PV_x of the previous tile is complete too: O_x is quiescent
        if (n_done > 0 && __any_sync(0xffffffffu, rescale)) {
          uint32_t oreg[32];
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            tmem_ld32(tO + c * 32, oreg);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) oreg[e] = __float_as_uint(__uint_as_float(oreg[e]) * corr);
            tmem_st32(tO + c * 32, oreg);
          }
        }
        // P as packed bf16 over the first 64 columns of S_x: column c holds keys 2c, 2c+1
        {
          uint32_t pk[32];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
#pragma unroll
            for (int e = 0; e < 16; ++e) { pk[e] = sreg[2 * h][e]; pk[16 + e] = sreg[2 * h + 1][e]; }
            tmem_st32(tS + h * 32, pk);
          }
        }
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive_warp(bar_p + x);
        ++n_done;
      }

      wait(bar_o, 0);
      tc_fence_after();
      const float inv_l = (l_sum > 0.f) ? 1.f / l_sum : 0.f;
      if (row < p.L) p.LSE[size_t(q_plane) * p.L + row] = (m_ref + log2f(l_sum)) * 0.6931471805599453f;
      __nv_bfloat16* orow = p.O + (size_t(q_plane) * p.L + row) * p.d;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
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
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
sepllm_status check_attn(const sepllm_attn_desc* d, const sepllm_index_desc* id) {
  if (!d || !id) return SEPLLM_INVALID_ARG;
  if (d->B <= 0 || d->Hq <= 0 || d->Hkv <= 0 || d->L <= 0 || d->Hq % d->Hkv != 0)
    return SEPLLM_INVALID_ARG;
  if (id->B != d->B || id->L != d->L || id->n_neighbor < 1 || id->n_init < 0 || id->side_cap <= 0)
    return SEPLLM_INVALID_ARG;
  if (d->d < 64 || d->d > 128 || d->d % 16 != 0) return SEPLLM_UNSUPPORTED;
  if (id->BM != kBM || id->BN != kBN) return SEPLLM_UNSUPPORTED;
  if (d->grad_dtype != 0 && d->grad_dtype != 1) return SEPLLM_INVALID_ARG;
  if (d->Hq > 65535 || d->B > 65535 || (d->L + kBM - 1) / kBM > 65535) return SEPLLM_UNSUPPORTED;
  return SEPLLM_OK;
}

AttnLayout attn_layout(const sepllm_attn_desc* d, const sepllm_index_desc* id) {
  AttnLayout a;
  a.cap_pad = (id->side_cap + 127) / 128 * 128;
  const int D = kernel_head_dim(d->d);
  const size_t side_bytes = align_up(size_t(d->B) * d->Hkv * a.cap_pad * D * 2);
  a.off_ks = kAlign;
  a.off_vs = a.off_ks + side_bytes;
  a.fwd_bytes = a.off_vs + side_bytes;
  a.off_delta = a.fwd_bytes;
  a.off_dks = a.off_delta + align_up(size_t(d->B) * d->Hq * d->L * 2 * sizeof(float));
  a.split = d->Hq / d->Hkv;  // one side-gradient partial per query head of a group
  const size_t side_grad =
      align_up(size_t(a.split) * d->B * d->Hkv * a.cap_pad * D * sizeof(float));
  a.off_dvs = a.off_dks + side_grad;
  a.bwd_bytes = a.off_dvs + side_grad;
  return a;
}

void launch_gather(const sepllm_attn_desc* d, const sepllm_index_desc* id, int cap_pad,
                   const void* K, const void* V, const int32_t* side_pos, const int32_t* n_side,
                   void* Ks, void* Vs, int32_t* status, cudaStream_t stream) {
  if (kernel_head_dim(d->d) == 64) {
    constexpr int RPB = 256 / (64 / 8);
    gather_side_kv<64><<<dim3((cap_pad + RPB - 1) / RPB, d->Hkv, d->B), 256, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(K), static_cast<const __nv_bfloat16*>(V), side_pos,
        n_side, d->L, d->d, d->Hkv, id->side_cap, cap_pad, static_cast<__nv_bfloat16*>(Ks),
        static_cast<__nv_bfloat16*>(Vs), status);
  } else {
    constexpr int RPB = 256 / (128 / 8);
    gather_side_kv<128><<<dim3((cap_pad + RPB - 1) / RPB, d->Hkv, d->B), 256, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(K), static_cast<const __nv_bfloat16*>(V), side_pos,
        n_side, d->L, d->d, d->Hkv, id->side_cap, cap_pad, static_cast<__nv_bfloat16*>(Ks),
        static_cast<__nv_bfloat16*>(Vs), status);
  }
}

template <int D>
static sepllm_status launch_fwd(const sepllm_attn_desc* d, const sepllm_index_desc* id,
                                const sepllm_index_header& ih, const void* Q, const void* K,
                                const void* V, const uint8_t* index, void* O, float* LSE,
                                uint8_t* ws, cudaStream_t stream) {
  const AttnLayout lay = attn_layout(d, id);
  __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(ws + lay.off_ks);
  __nv_bfloat16* Vs = reinterpret_cast<__nv_bfloat16*>(ws + lay.off_vs);
  const int32_t* side_pos = reinterpret_cast<const int32_t*>(index + ih.off_side_pos);
  const int32_t* n_side = reinterpret_cast<const int32_t*>(index + ih.off_n_side);
  record_event(d, 0, stream);
  if (!(d->flags & SEPLLM_ATTN_SIDE_READY))
    launch_gather(d, id, lay.cap_pad, K, V, side_pos, n_side, Ks, Vs, reinterpret_cast<int32_t*>(ws), stream);
  record_event(d, 1, stream);

  CUtensorMap mq, mk, mv, mks, mvs;
  sepllm_status st;
  const int64_t L = d->L, dr = d->d;  // rows of dr elements; the boxes read zeros from dr to D
  if ((st = make_tile_map(&mq, Q, dr, L, int64_t(d->B) * d->Hq, dr, L * dr, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mk, K, dr, L, int64_t(d->B) * d->Hkv, dr, L * dr, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mv, V, dr, L, int64_t(d->B) * d->Hkv, dr, L * dr, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mks, Ks, D, lay.cap_pad, int64_t(d->B) * d->Hkv, D,
                          int64_t(lay.cap_pad) * D, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mvs, Vs, D, lay.cap_pad, int64_t(d->B) * d->Hkv, D,
                          int64_t(lay.cap_pad) * D, 128)) != SEPLLM_OK) return st;

  FwdParams p;
  p.index_header = reinterpret_cast<const sepllm_index_header*>(index);
  p.cnt = reinterpret_cast<const int32_t*>(index + ih.off_cnt);
  p.lim = reinterpret_cast<const int32_t*>(index + ih.off_lim);
  p.tile_meta = reinterpret_cast<const int32_t*>(index + ih.off_tile_meta);
  p.seq_len = reinterpret_cast<const int32_t*>(index + ih.off_seq_len);
  p.doc_start = reinterpret_cast<const int32_t*>(index + ih.off_doc_start);
  p.doc_end = reinterpret_cast<const int32_t*>(index + ih.off_doc_end);
  p.O = static_cast<__nv_bfloat16*>(O);
  p.LSE = LSE;
  p.status = reinterpret_cast<int32_t*>(ws);
  p.L = d->L;
  p.d = d->d;
  p.T = ih.n_tiles;
  p.Hq = d->Hq;
  p.Hkv = d->Hkv;
  p.n_neighbor = id->n_neighbor;
  p.side_cap = id->side_cap;
  p.side_tiles_cap = lay.cap_pad / 128;
  const int G = d->Hq / d->Hkv;
  p.pair_heads = (G % 2 == 0) ? 1 : 0;
  const float scale = (d->scale != 0.f) ? d->scale : 1.0f / sqrtf(float(d->d));
  p.scale_log2 = scale * 1.4426950408889634f;
  if (D == 128 && G % 4 == 0) {
    // groups of four query heads: the CTA-pair kernel (K tiles loaded in 64-row halves)
    CUtensorMap mk64, mks64;
    if ((st = make_tile_map(&mk64, K, dr, L, int64_t(d->B) * d->Hkv, dr, L * dr, 64)) != SEPLLM_OK) return st;
    if ((st = make_tile_map(&mks64, Ks, D, lay.cap_pad, int64_t(d->B) * d->Hkv, D,
                            int64_t(lay.cap_pad) * D, 64)) != SEPLLM_OK) return st;
    st = launch_fwd_pair(d, p, ih.n_tiles, mq, mk64, mv, mks64, mvs, stream);
    record_event(d, 2, stream);
    return st;
  }
  const uint32_t smem = FwdCfg<D>::kRequest;
  SEPLLM_CUDA_TRY(cudaFuncSetAttribute(attn_fwd_kernel<D>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
  const dim3 grid = p.pair_heads ? dim3(d->Hq / 2 * d->B, ih.n_tiles)
                                 : dim3(d->Hq * d->B, (ih.n_tiles + 1) / 2);
  attn_fwd_kernel<D><<<grid, kFwdThreads, smem, stream>>>(mq, mk, mv, mks, mvs, p);
  record_event(d, 2, stream);
  SEPLLM_CUDA_TRY(cudaGetLastError());
  return SEPLLM_OK;
}

}  // namespace sepllm

using namespace sepllm;

extern "C" sepllm_status sepllm_attn_fwd(const sepllm_attn_desc* desc,
                                         const sepllm_index_desc* idesc, const void* Q,
                                         const void* K, const void* V, const void* index, void* O,
                                         float* LSE, void* workspace, void* stream_) {
  sepllm_status st = check_attn(desc, idesc);
  if (st != SEPLLM_OK) return st;
  if (!Q || !K || !V || !index || !O || !LSE || !workspace) return SEPLLM_INVALID_ARG;
  if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) ||
      !aligned(LSE, 4) || !aligned(index, kAlign) || !aligned(workspace, kAlign))
    return SEPLLM_INVALID_ARG;
  sepllm_index_header ih;
  if ((st = fill_index_header(idesc, &ih)) != SEPLLM_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  // (the side gather, the call's first launch, resets the status word)
  if (desc->flags & SEPLLM_ATTN_SIDE_READY) SEPLLM_CUDA_TRY(cudaMemsetAsync(ws, 0, sizeof(int32_t), stream));
  if (kernel_head_dim(desc->d) == 64)
    return launch_fwd<64>(desc, idesc, ih, Q, K, V, static_cast<const uint8_t*>(index), O, LSE, ws,
                          stream);
  return launch_fwd<128>(desc, idesc, ih, Q, K, V, static_cast<const uint8_t*>(index), O, LSE, ws,
                         stream);
}
