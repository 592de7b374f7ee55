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
#include "attn_common.cuh"

namespace sepllm {

constexpr float kLog2e = 1.4426950408889634f;

// ---------------------------------------------------------------------------
// Delta
// ---------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256)
bwd_delta(const __nv_bfloat16* __restrict__ dO, const __nv_bfloat16* __restrict__ O,
          float* __restrict__ delta, size_t rows) {
  constexpr int LPR = D / 8;
  const size_t r = (size_t(blockIdx.x) * 256 + threadIdx.x) / LPR;
  const int l = threadIdx.x % LPR;
  float s = 0.f;
  if (r < rows) {
    const uint4 a = *reinterpret_cast<const uint4*>(dO + r * D + l * 8);
    const uint4 b = *reinterpret_cast<const uint4*>(O + r * D + l * 8);
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
  if (r < rows && l == 0) delta[r] = s;
}

struct BwdParams {
  const int32_t* cnt;        // [B][L+1]
  const int32_t* lim;        // [B][L]
  const int32_t* side_pos;   // [B][side_cap]
  const int32_t* n_side;     // [B]
  const int32_t* tile_meta;  // [B][T][8]
  const float* LSE;          // [B][Hq][L]
  const float* delta;        // [B][Hq][L]
  float* dKs;                // [B][Hkv][cap_pad][D] fp32 side partials
  float* dVs;
  void* dQ;
  void* dK;
  void* dV;
  int32_t* status;
  int L, T, Hq, Hkv, n_neighbor, side_cap, cap_pad, grad_fp32;
  float scale, scale_log2;
};

__device__ __forceinline__ void store_row_chunk32(void* base, size_t elem_off, int fp32,
                                                  const float (&v)[32]) {
  if (fp32) {
    float4* dst = reinterpret_cast<float4*>(static_cast<float*>(base) + elem_off);
#pragma unroll
    for (int q = 0; q < 8; ++q) dst[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
  } else {
    uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(base) + elem_off);
#pragma unroll
    for (int q = 0; q < 4; ++q)
      dst[q] = make_uint4(pack_bf16(v[8 * q], v[8 * q + 1]), pack_bf16(v[8 * q + 2], v[8 * q + 3]),
                          pack_bf16(v[8 * q + 4], v[8 * q + 5]), pack_bf16(v[8 * q + 6], v[8 * q + 7]));
  }
}

// ---------------------------------------------------------------------------
// dQ: query-tile stationary
// ---------------------------------------------------------------------------
template <int D>
struct DqSmem {
  static constexpr int NB = D / 64;
  static constexpr uint32_t kQ = 0;
  static constexpr uint32_t kdO = kQ + NB * kTileBlockBytes;
  static constexpr uint32_t kK = kdO + NB * kTileBlockBytes;
  static constexpr uint32_t kV = kK + 2 * NB * kTileBlockBytes;
  static constexpr uint32_t kdS = kV + 2 * NB * kTileBlockBytes;
  static constexpr uint32_t kBar = kdS + 2 * kTileBlockBytes;
  static constexpr uint32_t kTotal = kBar + 256;
  static constexpr uint32_t kRequest = (kTotal + 1024 > 116 * 1024) ? kTotal + 1024 : 116 * 1024;
};

template <int D>
__global__ void __launch_bounds__(128, 1)
bwd_dq_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapdO,
              const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
              const __grid_constant__ CUtensorMap mapKs, const __grid_constant__ CUtensorMap mapVs,
              const BwdParams p) {
  using SM = DqSmem<D>;
  constexpr int NB = SM::NB;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~uintptr_t(1023));
  uint8_t* sQ = smem + SM::kQ;
  uint8_t* sdO = smem + SM::kdO;
  uint8_t* sK = smem + SM::kK;
  uint8_t* sV = smem + SM::kV;
  uint8_t* sdS = smem + SM::kdS;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::kBar);
  uint64_t* bar_q = bars + 0;
  uint64_t* bar_k = bars + 1;   // [2]
  uint64_t* bar_v = bars + 3;   // [2]
  uint64_t* bar_sp = bars + 5;  // S and dP of a tile are complete
  uint64_t* bar_dq = bars + 6;  // dQ MMA of a tile is complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 9);

  const int tid = threadIdx.x, warp = tid >> 5;
  const bool leader = (tid == 0);
  const int t = p.T - 1 - int(blockIdx.x);
  const int hq = blockIdx.y, b = blockIdx.z;
  const int G = p.Hq / p.Hkv;
  const int q_plane = b * p.Hq + hq;
  const int kv_plane = b * p.Hkv + hq / G;

  if (leader) {
    mbar_init(bar_q, 1);
    for (int i = 0; i < 2; ++i) { mbar_init(bar_k + i, 1); mbar_init(bar_v + i, 1); }
    mbar_init(bar_sp, 1);
    mbar_init(bar_dq, 1);
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
  const uint32_t tmem_row = tmem + (uint32_t(warp * 32) << 16);
  constexpr uint32_t tmem_S = 0, tmem_dP = 128, tmem_dQ = 256;

  const int32_t* meta = p.tile_meta + (size_t(b) * p.T + t) * 8;
  const int side_full = meta[0];
  const int n_side_tiles = min(meta[1], p.cap_pad / kBN);
  const int win_tile_lo = meta[4];
  const int n_tiles = n_side_tiles + (meta[5] - win_tile_lo);
  const int row = t * kBM + tid;
  const bool row_ok = row < p.L;
  const int lim_i = row_ok ? min(p.lim[size_t(b) * p.L + row], p.side_cap) : 0;
  const float lse2 = row_ok ? p.LSE[size_t(q_plane) * p.L + row] * kLog2e : INFINITY;
  const float delta_i = row_ok ? p.delta[size_t(q_plane) * p.L + row] : 0.f;

  auto tile_y = [&](int j) {
    return (j < n_side_tiles) ? j * kBN : (win_tile_lo + (j - n_side_tiles)) * kBN;
  };
  auto load_k = [&](int j) {
    const int st = j & 1;
    mbar_expect_tx(bar_k + st, NB * kTileBlockBytes);
    for (int nb = 0; nb < NB; ++nb)
      tma_load_3d(sK + (st * NB + nb) * kTileBlockBytes, (j < n_side_tiles) ? &mapKs : &mapK,
                  bar_k + st, nb * 64, tile_y(j), kv_plane);
  };
  auto load_v = [&](int j) {
    const int st = j & 1;
    mbar_expect_tx(bar_v + st, NB * kTileBlockBytes);
    for (int nb = 0; nb < NB; ++nb)
      tma_load_3d(sV + (st * NB + nb) * kTileBlockBytes, (j < n_side_tiles) ? &mapVs : &mapV,
                  bar_v + st, nb * 64, tile_y(j), kv_plane);
  };
  bool ok = true;
  auto wait = [&](uint64_t* bar, uint32_t parity) {
    if (!mbar_wait(bar, parity, abort_flag)) {
      if (ok) set_status(p.status, SEPLLM_TIMEOUT);
      ok = false;
    }
  };
  constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);
  constexpr uint32_t idesc_dq = make_idesc_bf16(128, D, 0, 1);

  if (leader) {
    mbar_expect_tx(bar_q, 2 * NB * kTileBlockBytes);
    for (int nb = 0; nb < NB; ++nb) {
      tma_load_3d(sQ + nb * kTileBlockBytes, &mapQ, bar_q, nb * 64, t * kBM, q_plane);
      tma_load_3d(sdO + nb * kTileBlockBytes, &mapdO, bar_q, nb * 64, t * kBM, q_plane);
    }
    load_k(0);
    load_v(0);
    if (n_tiles > 1) { load_k(1); load_v(1); }
    wait(bar_q, 0);
  }

  for (int j = 0; j < n_tiles; ++j) {
    const int st = j & 1;
    if (leader) {
      const uint32_t qa = smem_u32(sQ), doa = smem_u32(sdO);
      const uint32_t ka = smem_u32(sK + st * NB * kTileBlockBytes);
      const uint32_t va = smem_u32(sV + st * NB * kTileBlockBytes);
      wait(bar_k + st, (j >> 1) & 1);
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < D / 16; ++k) {
        const uint32_t off = (k / 4) * kTileBlockBytes + (k % 4) * 32;
        umma_ss(tmem + tmem_S, make_smem_desc(qa + off, 16, 1024), make_smem_desc(ka + off, 16, 1024),
                idesc_s, k > 0);
      }
      wait(bar_v + st, (j >> 1) & 1);
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < D / 16; ++k) {
        const uint32_t off = (k / 4) * kTileBlockBytes + (k % 4) * 32;
        umma_ss(tmem + tmem_dP, make_smem_desc(doa + off, 16, 1024),
                make_smem_desc(va + off, 16, 1024), idesc_s, k > 0);
      }
      tc_commit(bar_sp);
    }
    wait(bar_sp, j & 1);
    tc_fence_after();
    if (leader && j + 2 < n_tiles) load_v(j + 2);  // dP(j) is complete: its V stage is free
    __syncwarp();

    const bool side = j < n_side_tiles;
    int c_lo = 0, c_hi = kBN;
    bool need_mask;
    if (side) {
      c_hi = lim_i - j * kBN;
      need_mask = (j >= side_full);
    } else {
      const int key0 = tile_y(j);
      c_hi = row - key0 + 1;
      c_lo = row - p.n_neighbor + 1 - key0;
      need_mask = (key0 + kBN - 1 > t * kBM) || (key0 < t * kBM + kBM - p.n_neighbor);
    }
    // dQ MMA of the previous tile reads sdS and its K stage
    if (j > 0) {
      wait(bar_dq, (j - 1) & 1);
      tc_fence_after();
      if (leader && j + 1 < n_tiles && j >= 1) {
        if (j + 1 >= 2) load_k(j + 1);  // K stage of tile j-1 is free now
      }
    }
    __syncwarp();
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      uint32_t s[32], dp[32];
      tmem_ld32(tmem_row + tmem_S + c * 32, s);
      tmem_ld32(tmem_row + tmem_dP + c * 32, dp);
      tmem_ld_wait();
#pragma unroll
      for (int e = 0; e < 32; e += 2) {
        float ds[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int col = c * 32 + e + u;
          float pr = ex2(__uint_as_float(s[e + u]) * p.scale_log2 - lse2);
          if (need_mask && !(col >= c_lo && col < c_hi)) pr = 0.f;
          ds[u] = pr * (__uint_as_float(dp[e + u]) - delta_i);
        }
        s[e >> 1] = pack_bf16(ds[0], ds[1]);
      }
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        const int chunk16 = c * 4 + q4;
        *reinterpret_cast<uint4*>(sdS + (chunk16 >> 3) * kTileBlockBytes + swz128(tid, chunk16 & 7)) =
            make_uint4(s[q4 * 4], s[q4 * 4 + 1], s[q4 * 4 + 2], s[q4 * 4 + 3]);
      }
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    if (leader) {
      tc_fence_after();
      const uint32_t dsa = smem_u32(sdS), ka = smem_u32(sK + st * NB * kTileBlockBytes);
#pragma unroll
      for (int k = 0; k < kBN / 16; ++k) {
        const uint32_t aoff = (k / 4) * kTileBlockBytes + (k % 4) * 32;
        umma_ss(tmem + tmem_dQ, make_smem_desc(dsa + aoff, 16, 1024),
                make_smem_desc(ka + k * 2048, kTileBlockBytes, 1024), idesc_dq, (j > 0 || k > 0));
      }
      tc_commit(bar_dq);
    }
  }

  wait(bar_dq, (n_tiles - 1) & 1);
  tc_fence_after();
  __syncwarp();
#pragma unroll
  for (int c = 0; c < D / 32; ++c) {
    uint32_t r[32];
    tmem_ld32(tmem_row + tmem_dQ + c * 32, r);
    tmem_ld_wait();
    if (row_ok) {
      float v[32];
#pragma unroll
      for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(r[e]) * p.scale;
      store_row_chunk32(p.dQ, (size_t(q_plane) * p.L + row) * D + c * 32, p.grad_fp32, v);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

// ---------------------------------------------------------------------------
// dK, dV: key-tile stationary
// ---------------------------------------------------------------------------
template <int D>
struct DkvSmem {
  static constexpr int NB = D / 64;
  static constexpr uint32_t kK = 0;
  static constexpr uint32_t kV = kK + NB * kTileBlockBytes;
  static constexpr uint32_t kQ = kV + NB * kTileBlockBytes;
  static constexpr uint32_t kdO = kQ + NB * kTileBlockBytes;
  static constexpr uint32_t kPT = kdO + NB * kTileBlockBytes;
  static constexpr uint32_t kdST = kPT + 2 * kTileBlockBytes;
  static constexpr uint32_t kRow = kdST + 2 * kTileBlockBytes;  // lse2[128], delta[128], lim[128]
  static constexpr uint32_t kBar = kRow + 3 * 128 * 4;
  static constexpr uint32_t kTotal = kBar + 256;
  static constexpr uint32_t kRequest = (kTotal + 1024 > 116 * 1024) ? kTotal + 1024 : 116 * 1024;
};

template <int D, bool SIDE>
__global__ void __launch_bounds__(128, 1)
bwd_dkv_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapdO,
               const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
               const BwdParams p) {
  using SM = DkvSmem<D>;
  constexpr int NB = SM::NB;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~uintptr_t(1023));
  uint8_t* sK = smem + SM::kK;
  uint8_t* sV = smem + SM::kV;
  uint8_t* sQ = smem + SM::kQ;
  uint8_t* sdO = smem + SM::kdO;
  uint8_t* sPT = smem + SM::kPT;
  uint8_t* sdST = smem + SM::kdST;
  float* s_lse2 = reinterpret_cast<float*>(smem + SM::kRow);
  float* s_delta = s_lse2 + 128;
  int32_t* s_lim = reinterpret_cast<int32_t*>(s_delta + 128);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::kBar);
  uint64_t* bar_kv = bars + 0;
  uint64_t* bar_qdo = bars + 1;
  uint64_t* bar_sp = bars + 2;
  uint64_t* bar_acc = bars + 3;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 9);

  const int tid = threadIdx.x, warp = tid >> 5;
  const bool leader = (tid == 0);
  const int kt = SIDE ? int(blockIdx.x) : int(gridDim.x) - 1 - int(blockIdx.x);
  const int hk = blockIdx.y, b = blockIdx.z;
  const int G = p.Hq / p.Hkv;
  const int kv_plane = b * p.Hkv + hk;
  const int ns = min(p.n_side[b], p.side_cap);

  // query tiles that keep at least one key of this tile
  int t_lo, t_hi;
  if (SIDE) {
    if (kt * kBN >= ns) return;  // no entries in this side tile: nothing reads its partial rows
    t_lo = (p.side_pos[size_t(b) * p.side_cap + kt * kBN] + p.n_neighbor) / kBM;
    t_hi = p.T - 1;
  } else {
    t_lo = kt;  // kBM == kBN
    t_hi = min(p.T - 1, (kt * kBN + kBN - 1 + p.n_neighbor - 1) / kBM);
  }
  const int n_qt = max(0, t_hi - t_lo + 1);
  const int n_iter = n_qt * G;

  if (leader) {
    mbar_init(bar_kv, 1);
    mbar_init(bar_qdo, 1);
    mbar_init(bar_sp, 1);
    mbar_init(bar_acc, 1);
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
  const uint32_t tmem_row = tmem + (uint32_t(warp * 32) << 16);
  constexpr uint32_t tmem_ST = 0, tmem_dPT = 128, tmem_dV = 256, tmem_dK = 256 + D;

  bool ok = true;
  auto wait = [&](uint64_t* bar, uint32_t parity) {
    if (!mbar_wait(bar, parity, abort_flag)) {
      if (ok) set_status(p.status, SEPLLM_TIMEOUT);
      ok = false;
    }
  };
  auto load_qdo = [&](int it) {
    const int tq = t_lo + it / G, g = it % G;
    const int q_plane = b * p.Hq + hk * G + g;
    mbar_expect_tx(bar_qdo, 2 * NB * kTileBlockBytes);
    for (int nb = 0; nb < NB; ++nb) {
      tma_load_3d(sQ + nb * kTileBlockBytes, &mapQ, bar_qdo, nb * 64, tq * kBM, q_plane);
      tma_load_3d(sdO + nb * kTileBlockBytes, &mapdO, bar_qdo, nb * 64, tq * kBM, q_plane);
    }
  };
  constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);
  constexpr uint32_t idesc_acc = make_idesc_bf16(128, D, 0, 1);

  if (leader && n_iter > 0) {
    mbar_expect_tx(bar_kv, 2 * NB * kTileBlockBytes);
    for (int nb = 0; nb < NB; ++nb) {
      tma_load_3d(sK + nb * kTileBlockBytes, &mapK, bar_kv, nb * 64, kt * kBN, kv_plane);
      tma_load_3d(sV + nb * kTileBlockBytes, &mapV, bar_kv, nb * 64, kt * kBN, kv_plane);
    }
    load_qdo(0);
    wait(bar_kv, 0);
  }

  const int key = kt * kBN + tid;  // side entry index (SIDE) or key position (window)

  for (int it = 0; it < n_iter; ++it) {
    const int tq = t_lo + it / G, g = it % G;
    const int q_plane = b * p.Hq + hk * G + g;
    if (it > 0) {
      // dV/dK MMAs of the previous iteration read sQ, sdO, sPT, sdST
      wait(bar_acc, (it - 1) & 1);
      tc_fence_after();
      if (leader) load_qdo(it);
    }
    __syncthreads();  // previous readers of the per-row arrays are done
    {
      const int qi = tq * kBM + tid;
      const bool q_ok = qi < p.L;
      s_lse2[tid] = q_ok ? p.LSE[size_t(q_plane) * p.L + qi] * kLog2e : INFINITY;
      s_delta[tid] = q_ok ? p.delta[size_t(q_plane) * p.L + qi] : 0.f;
      if (SIDE) s_lim[tid] = q_ok ? min(p.lim[size_t(b) * p.L + qi], p.side_cap) : 0x7fffffff;
    }
    if (leader) {
      wait(bar_qdo, it & 1);
      tc_fence_after();
      const uint32_t ka = smem_u32(sK), va = smem_u32(sV), qa = smem_u32(sQ), doa = smem_u32(sdO);
#pragma unroll
      for (int k = 0; k < D / 16; ++k) {
        const uint32_t off = (k / 4) * kTileBlockBytes + (k % 4) * 32;
        umma_ss(tmem + tmem_ST, make_smem_desc(ka + off, 16, 1024), make_smem_desc(qa + off, 16, 1024),
                idesc_s, k > 0);
      }
#pragma unroll
      for (int k = 0; k < D / 16; ++k) {
        const uint32_t off = (k / 4) * kTileBlockBytes + (k % 4) * 32;
        umma_ss(tmem + tmem_dPT, make_smem_desc(va + off, 16, 1024),
                make_smem_desc(doa + off, 16, 1024), idesc_s, k > 0);
      }
      tc_commit(bar_sp);
    }
    __syncthreads();  // per-row arrays are written

    // kept query columns for this key row: [q_lo, q_hi)
    int q_lo, q_hi = kBM;
    bool need_mask;
    if (SIDE) {
      // lim is non-decreasing: kept from the first query with lim > key
      int lo = 0, hi = kBM;
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (s_lim[mid] > key) hi = mid; else lo = mid + 1;
      }
      q_lo = lo;
      need_mask = true;
    } else {
      q_lo = key - tq * kBM;
      q_hi = key + p.n_neighbor - tq * kBM;
      need_mask = true;
    }
    wait(bar_sp, it & 1);
    tc_fence_after();
    __syncwarp();
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      uint32_t s[32], dp[32];
      tmem_ld32(tmem_row + tmem_ST + c * 32, s);
      tmem_ld32(tmem_row + tmem_dPT + c * 32, dp);
      tmem_ld_wait();
#pragma unroll
      for (int e = 0; e < 32; e += 2) {
        float pr[2], ds[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int col = c * 32 + e + u;
          pr[u] = ex2(__uint_as_float(s[e + u]) * p.scale_log2 - s_lse2[col]);
          if (need_mask && !(col >= q_lo && col < q_hi)) pr[u] = 0.f;
          ds[u] = pr[u] * (__uint_as_float(dp[e + u]) - s_delta[col]);
        }
        s[e >> 1] = pack_bf16(pr[0], pr[1]);
        dp[e >> 1] = pack_bf16(ds[0], ds[1]);
      }
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        const int chunk16 = c * 4 + q4;
        const uint32_t off = (chunk16 >> 3) * kTileBlockBytes + swz128(tid, chunk16 & 7);
        *reinterpret_cast<uint4*>(sPT + off) = make_uint4(s[q4 * 4], s[q4 * 4 + 1], s[q4 * 4 + 2], s[q4 * 4 + 3]);
        *reinterpret_cast<uint4*>(sdST + off) = make_uint4(dp[q4 * 4], dp[q4 * 4 + 1], dp[q4 * 4 + 2], dp[q4 * 4 + 3]);
      }
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    if (leader) {
      tc_fence_after();
      const uint32_t pta = smem_u32(sPT), dsta = smem_u32(sdST), qa = smem_u32(sQ), doa = smem_u32(sdO);
#pragma unroll
      for (int k = 0; k < kBM / 16; ++k) {
        const uint32_t aoff = (k / 4) * kTileBlockBytes + (k % 4) * 32;
        umma_ss(tmem + tmem_dV, make_smem_desc(pta + aoff, 16, 1024),
                make_smem_desc(doa + k * 2048, kTileBlockBytes, 1024), idesc_acc, (it > 0 || k > 0));
      }
#pragma unroll
      for (int k = 0; k < kBM / 16; ++k) {
        const uint32_t aoff = (k / 4) * kTileBlockBytes + (k % 4) * 32;
        umma_ss(tmem + tmem_dK, make_smem_desc(dsta + aoff, 16, 1024),
                make_smem_desc(qa + k * 2048, kTileBlockBytes, 1024), idesc_acc, (it > 0 || k > 0));
      }
      tc_commit(bar_acc);
    }
  }

  if (n_iter > 0) {
    wait(bar_acc, (n_iter - 1) & 1);
    tc_fence_after();
  }
  __syncwarp();

  if (SIDE) {
    // fp32 partial rows for the entries of this side tile
    const bool r_ok = key < p.cap_pad;
    float* dks = p.dKs + (size_t(kv_plane) * p.cap_pad + key) * D;
    float* dvs = p.dVs + (size_t(kv_plane) * p.cap_pad + key) * D;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
      uint32_t rk[32], rv[32];
      if (n_iter > 0) {
        tmem_ld32(tmem_row + tmem_dK + c * 32, rk);
        tmem_ld32(tmem_row + tmem_dV + c * 32, rv);
        tmem_ld_wait();
      } else {
#pragma unroll
        for (int e = 0; e < 32; ++e) { rk[e] = 0; rv[e] = 0; }
      }
      if (r_ok) {
        float v[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(rk[e]) * p.scale;
        store_row_chunk32(dks, c * 32, 1, v);
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(rv[e]);
        store_row_chunk32(dvs, c * 32, 1, v);
      }
    }
  } else {
    // final rows: window part plus, for initial/separator tokens, the side partial of the same token
    const bool r_ok = key < p.L;
    int side_idx = -1;
    if (r_ok) {
      const int32_t* cnt_b = p.cnt + size_t(b) * (p.L + 1);
      const int c0 = cnt_b[key], c1 = cnt_b[key + 1];
      if (c1 > c0 && c0 < ns) {
        // the side pass wrote this row only if some query sees it from outside its window
        const int t_first = (key + p.n_neighbor) / kBM;
        if (t_first <= p.T - 1) side_idx = c0;
      }
    }
    const float* dks = p.dKs + (size_t(kv_plane) * p.cap_pad + max(side_idx, 0)) * D;
    const float* dvs = p.dVs + (size_t(kv_plane) * p.cap_pad + max(side_idx, 0)) * D;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
      uint32_t rk[32], rv[32];
      tmem_ld32(tmem_row + tmem_dK + c * 32, rk);
      tmem_ld32(tmem_row + tmem_dV + c * 32, rv);
      tmem_ld_wait();
      if (r_ok) {
        float v[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(rk[e]) * p.scale;
        if (side_idx >= 0) {
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] += dks[c * 32 + e];
        }
        store_row_chunk32(p.dK, (size_t(kv_plane) * p.L + key) * D + c * 32, p.grad_fp32, v);
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(rv[e]);
        if (side_idx >= 0) {
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] += dvs[c * 32 + e];
        }
        store_row_chunk32(p.dV, (size_t(kv_plane) * p.L + key) * D + c * 32, p.grad_fp32, v);
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
    launch_gather(d, id, lay.cap_pad, K, V, side_pos, n_side, Ks, Vs, stream);
  record_event(d, 1, stream);

  float* delta = reinterpret_cast<float*>(ws + lay.off_delta);
  const size_t rows = size_t(d->B) * d->Hq * d->L;
  {
    constexpr int RPB = 256 / (D / 8);
    bwd_delta<D><<<unsigned((rows + RPB - 1) / RPB), 256, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(dO), static_cast<const __nv_bfloat16*>(O), delta, rows);
  }
  record_event(d, 2, stream);

  CUtensorMap mq, mdo, mk, mv, mks, mvs;
  sepllm_status st;
  const int64_t L = d->L;
  if ((st = make_tile_map(&mq, Q, D, L, int64_t(d->B) * d->Hq, D, L * D, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mdo, dO, D, L, int64_t(d->B) * d->Hq, D, L * D, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mk, K, D, L, int64_t(d->B) * d->Hkv, D, L * D, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mv, V, D, L, int64_t(d->B) * d->Hkv, D, L * D, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mks, Ks, D, lay.cap_pad, int64_t(d->B) * d->Hkv, D,
                          int64_t(lay.cap_pad) * D, 128)) != SEPLLM_OK) return st;
  if ((st = make_tile_map(&mvs, Vs, D, lay.cap_pad, int64_t(d->B) * d->Hkv, D,
                          int64_t(lay.cap_pad) * D, 128)) != SEPLLM_OK) return st;

  BwdParams p;
  p.cnt = reinterpret_cast<const int32_t*>(index + ih.off_cnt);
  p.lim = reinterpret_cast<const int32_t*>(index + ih.off_lim);
  p.side_pos = side_pos;
  p.n_side = n_side;
  p.tile_meta = reinterpret_cast<const int32_t*>(index + ih.off_tile_meta);
  p.LSE = LSE;
  p.delta = delta;
  p.dKs = reinterpret_cast<float*>(ws + lay.off_dks);
  p.dVs = reinterpret_cast<float*>(ws + lay.off_dvs);
  p.dQ = dQ;
  p.dK = dK;
  p.dV = dV;
  p.status = reinterpret_cast<int32_t*>(ws);
  p.L = d->L;
  p.T = ih.n_tiles;
  p.Hq = d->Hq;
  p.Hkv = d->Hkv;
  p.n_neighbor = id->n_neighbor;
  p.side_cap = id->side_cap;
  p.cap_pad = lay.cap_pad;
  p.grad_fp32 = d->grad_dtype;
  p.scale = (d->scale != 0.f) ? d->scale : 1.0f / sqrtf(float(D));
  p.scale_log2 = p.scale * kLog2e;

  SEPLLM_CUDA_TRY(cudaFuncSetAttribute(bwd_dq_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       int(DqSmem<D>::kRequest)));
  SEPLLM_CUDA_TRY(cudaFuncSetAttribute(bwd_dkv_kernel<D, true>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       int(DkvSmem<D>::kRequest)));
  SEPLLM_CUDA_TRY(cudaFuncSetAttribute(bwd_dkv_kernel<D, false>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       int(DkvSmem<D>::kRequest)));
  bwd_dq_kernel<D><<<dim3(ih.n_tiles, d->Hq, d->B), 128, DqSmem<D>::kRequest, stream>>>(
      mq, mdo, mk, mv, mks, mvs, p);
  record_event(d, 3, stream);
  bwd_dkv_kernel<D, true><<<dim3(lay.cap_pad / kBN, d->Hkv, d->B), 128, DkvSmem<D>::kRequest,
                            stream>>>(mq, mdo, mks, mvs, p);
  record_event(d, 4, stream);
  bwd_dkv_kernel<D, false><<<dim3(ih.n_tiles, d->Hkv, d->B), 128, DkvSmem<D>::kRequest, stream>>>(
      mq, mdo, mk, mv, p);
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
  SEPLLM_CUDA_TRY(cudaMemsetAsync(ws, 0, kAlign, stream));
  const uint8_t* idx = static_cast<const uint8_t*>(index);
  if (desc->d == 64)
    return launch_bwd<64>(desc, idesc, ih, dO, Q, K, V, O, LSE, idx, dQ, dK, dV, ws, stream);
  return launch_bwd<128>(desc, idesc, ih, dO, Q, K, V, O, LSE, idx, dQ, dK, dV, ws, stream);
}
