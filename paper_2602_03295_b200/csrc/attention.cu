// Causal, GQA-aware flash-attention prefill on tcgen05 (the Attn(x_l, K, V) of paper Eq. 1, reading
// the cache that Eq. 2-3 just filled), with an optional sliding window.
//
// One CTA owns 128 consecutive query positions of NQT query heads that share a KV head (NQT = 2
// when the GQA ratio allows it: both tiles see the same keys and the same mask, so every K/V
// tile staged in shared memory is used twice). Keys are walked 64 at a time. Warp roles:
//   NQT softmax warpgroups (128 threads each, one query row per thread): read S = Q K^T from one
//       of two TMEM score buffers, keep the running row maximum / sum in fp32, write
//       P = exp2(S - m) as packed bf16 over the front half of the same buffer (the tensor core
//       reads the A operand of P V straight from TMEM), rescale the O accumulator in TMEM only
//       when the maximum grew by more than 2^8, and finally normalise and store O;
//   1 TMA warp: Q tiles once, then K and V tiles of the paged cache through a deep ring of
//       shared-memory stages (no shared memory is spent on P: the latency of fetching scattered
//       cache rows is what has to be hidden);
//   1 MMA warp: allocates TMEM and keeps the scores two key tiles ahead of the softmax: when
//       P_t of tile j is ready it issues O_t += P_t V_j and, behind it, S_t = Q_t K_{j+2}^T into the
//       buffer P_t just vacated, so a softmax warpgroup never waits for the tensor pipe's latency.
// K/V come straight from the paged cache [page][slot][kv head][hd] with 4-D tensor maps; cache
// positions >= kv_len are never dereferenced through the block table and never reach the output.
#include "common.cuh"
#include "ptx.cuh"

#include <type_traits>

namespace pop {
namespace {

constexpr int kSmemLimit = 227 * 1024;

template <int HD, int NQT>
struct AC {
  static constexpr int BKV = 64;
  static constexpr int KV_TILE_BYTES = BKV * HD * 2;
  static constexpr int KV_SUB_BYTES = BKV * 128;     // one 64-wide slice of head_dim
  static constexpr int Q_TILE_BYTES = 128 * HD * 2;
  static constexpr int RING_BYTES = kSmemLimit - 3 * 1024 - NQT * Q_TILE_BYTES;   // alignment slack + barriers
  static constexpr int STAGES = RING_BYTES / KV_TILE_BYTES < 12 ? RING_BYTES / KV_TILE_BYTES : 12;
  static constexpr int THREADS = NQT * 128 + 64;
  // TMEM columns: two score buffers per tile (P overwrites the first 32 columns of the buffer its
  // scores came from), then the output accumulators
  static constexpr int S_COL = 0;                    // S_t[b] at (t * 2 + b) * 64
  static constexpr int O_COL = NQT * 2 * BKV;        // O_t at O_COL + t * HD
  static constexpr int COLS_USED = O_COL + NQT * HD;
  static constexpr uint32_t TMEM_COLS = COLS_USED <= 128 ? 128 : (COLS_USED <= 256 ? 256 : 512);
  static_assert(COLS_USED <= 512, "TMEM budget");
  static_assert(STAGES >= 4, "ring too shallow");
};

template <int HD, int NQT>
struct __align__(1024) AttnSmem {
  using C = AC<HD, NQT>;
  uint8_t q[NQT][C::Q_TILE_BYTES];
  uint8_t kv[C::STAGES][C::KV_TILE_BYTES];
  uint64_t q_full;
  uint64_t kv_full[C::STAGES];
  uint64_t kv_empty[C::STAGES];
  // one barrier per tile and score buffer b = key tile & 1; phase = key tile >> 1. Producer and
  // consumer of one buffer alternate strictly, so a parity wait is never two phases behind.
  uint64_t s_full[NQT][2];      // S_t[b] = Q_t K^T complete
  uint64_t p_ready[NQT][2];     // P_t[b] written over S_t[b] (one arrival per softmax warp)
  uint64_t pv_done[NQT][2];     // O_t += P_t[b] V complete
  uint32_t tmem_base;
  uint32_t raised;
  volatile uint32_t abort;
};

struct AttnDev {
  bf16* out;            // [batch*seq][ldo]
  int64_t ldo;
  const int32_t* block_table;
  int max_pages_per_seq;
  int page_size;
  int rows_per_load;    // min(page_size, BKV)
  int seq_len;          // query rows per sequence (positions q_pos0 .. q_pos0 + seq_len - 1)
  int q_pos0;
  int kv_len;           // valid cache positions per sequence
  int n_q_heads, n_kv_heads;
  int window;
  int num_pages;        // block-table entries are checked against it
  int q_tiles;
  float scale_log2;     // log2(e) / sqrt(hd)
  const int32_t* cu;    // ragged batches: packed-row prefix sums [batch + 1], or null
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

#define POP_ABORT(S, status)                          \
  do {                                                \
    (S).abort = 1;                                    \
    atomicMin((status), (int)POP_E_DEVICE_TIMEOUT);   \
  } while (0)

template <int HD, int NQT>
__global__ void __launch_bounds__(AC<HD, NQT>::THREADS, 1)
attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
            const __grid_constant__ CUtensorMap tmV, const AttnDev p, int* __restrict__ status) {
  using C = AC<HD, NQT>;
  constexpr int BKV = C::BKV;
  constexpr int STAGES = C::STAGES;
  extern __shared__ uint8_t smem_raw[];
  AttnSmem<HD, NQT>& s =
      *reinterpret_cast<AttnSmem<HD, NQT>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  // heaviest query tiles (latest positions) first
  const int q_tile = p.q_tiles - 1 - (int)blockIdx.y;
  const int head0 = blockIdx.x * NQT;
  const int b = blockIdx.z;
  const int kv_head = head0 * p.n_kv_heads / p.n_q_heads;
  const int q_row0 = q_tile * 128;                       // row within the sequence
  // a ragged batch gives every sequence its own length; query tiles past its end have nothing to do
  const int row_base = p.cu ? p.cu[b] : b * p.seq_len;   // first packed row of the sequence
  const int seq_len = p.cu ? p.cu[b + 1] - row_base : p.seq_len;
  const int kv_len = p.cu ? seq_len : p.kv_len;
  if (q_row0 >= seq_len) return;
  const int pos0 = p.q_pos0 + q_row0;                    // absolute position of row 0
  const int last_pos = min(pos0 + 127, p.q_pos0 + seq_len - 1);
  const int j_hi = min(last_pos, kv_len - 1) / BKV;
  const int j_lo = p.window > 0 ? max(0, pos0 - p.window + 1) / BKV : 0;
  const int n_tiles = j_hi - j_lo + 1;

  if (status_raised(status, &s.raised)) return;
  if (threadIdx.x == 0) {
    mbar_init(&s.q_full, 1);
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(&s.kv_full[i], 1);
      mbar_init(&s.kv_empty[i], 1);
    }
    for (int t = 0; t < NQT; ++t)
      for (int i = 0; i < 2; ++i) {
        mbar_init(&s.s_full[t][i], 1);
        mbar_init(&s.p_ready[t][i], 4);
        mbar_init(&s.pv_done[t][i], 1);
      }
    s.abort = 0;
    fence_barrier_init();
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
  }
  if (warp == NQT * 4 + 1) {
    tmem_alloc(&s.tmem_base, C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s.tmem_base;

  if (warp == NQT * 4) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(&s.q_full, NQT * C::Q_TILE_BYTES);
      for (int t = 0; t < NQT; ++t)
        for (int c = 0; c < HD / 64; ++c)
          tma_load_3d(s.q[t] + c * 16384, &tmQ, &s.q_full, c * 64, head0 + t, row_base + q_row0);
      const int32_t* bt = p.block_table + (int64_t)b * p.max_pages_per_seq;
      const int loads_per_tile = BKV / p.rows_per_load;
      // ring order = the order the MMA warp consumes: K_0, K_1, then V_j, K_{j+2} for j = 0, 1, ...
      int ring = 0;
      bool ok = true;
      auto load_tile = [&](int j, const CUtensorMap* tm) {
        const int kv0 = (j_lo + j) * BKV;
        const int stage = ring % STAGES;
        const uint32_t phase = (ring / STAGES) & 1;
        ++ring;
        if (!mbar_wait_relaxed(&s.kv_empty[stage], phase ^ 1)) {
          POP_ABORT(s, status);
          ok = false;
          return;
        }
        int n_loads = 0;
        for (int r = 0; r < loads_per_tile; ++r)
          if (kv0 + r * p.rows_per_load < kv_len) ++n_loads;
        mbar_expect_tx(&s.kv_full[stage], n_loads * p.rows_per_load * HD * 2);
        for (int r = 0; r < n_loads; ++r) {
          const int pos = kv0 + r * p.rows_per_load;
          const int page = bt[pos / p.page_size];
          // an entry outside the pool cannot fault here (the tensor map clips), but it is an error
          if ((unsigned)page >= (unsigned)p.num_pages) atomicMin(status, (int)POP_E_INVALID);
          const int slot = pos % p.page_size;
          for (int c = 0; c < HD / 64; ++c)
            tma_load_4d(s.kv[stage] + c * C::KV_SUB_BYTES + r * p.rows_per_load * 128, tm, &s.kv_full[stage],
                        c * 64, kv_head, slot, page);
        }
      };
      load_tile(0, &tmK);
      if (ok && n_tiles > 1) load_tile(1, &tmK);
      for (int jj = 0; jj < n_tiles && ok && !s.abort; ++jj) {
        load_tile(jj, &tmV);
        if (ok && jj + 2 < n_tiles) load_tile(jj + 2, &tmK);
      }
    }
  } else if (warp == NQT * 4 + 1) {
    // ------------------------------------------------------------------ MMA issuer
    {
      // the whole warp walks this role; one elected lane issues the tensor-core instructions
      const uint32_t leader = elect_one();
      constexpr uint32_t idesc_s = umma_idesc_bf16(128, BKV, 0, 0);
      constexpr uint32_t idesc_o = umma_idesc_bf16(128, HD, 0, 1);
      // Operand descriptors are built once; per instruction only the 16-byte-granular start address
      // in the low bits moves (all shared-memory offsets here stay far below the field's 256 KB).
      uint64_t q_desc[NQT];
      for (int t = 0; t < NQT; ++t) q_desc[t] = umma_smem_desc(smem_u32(s.q[t]), 16, 1024);
      const uint64_t k_desc0 = umma_smem_desc(smem_u32(s.kv[0]), 16, 1024);                 // K-major
      const uint64_t v_desc0 = umma_smem_desc(smem_u32(s.kv[0]), C::KV_SUB_BYTES, 1024);    // MN-major
      auto issue_s = [&](int t, int j, int stage) {
        const uint64_t qd = q_desc[t];
        const uint64_t kd = k_desc0 + uint64_t(stage * (C::KV_TILE_BYTES >> 4));
        const uint32_t d = tmem_base + C::S_COL + (t * 2 + (j & 1)) * BKV;
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          const uint64_t ad = qd + uint64_t(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
          const uint64_t bd = kd + uint64_t(((kk >> 2) * C::KV_SUB_BYTES + (kk & 3) * 32) >> 4);
          umma_bf16_ss_w(leader, d, ad, bd, idesc_s, kk > 0 ? 1u : 0u);
        }
        umma_commit_w(leader, &s.s_full[t][j & 1]);
      };
      auto issue_pv = [&](int t, int j, int stage) {
        // A operand = P_t in TMEM: 16 keys are 8 packed 32-bit columns; B = V tile, MN-major
        const uint32_t pa = tmem_base + C::S_COL + (t * 2 + (j & 1)) * BKV;
        const uint64_t vd = v_desc0 + uint64_t(stage * (C::KV_TILE_BYTES >> 4));
        const uint32_t d = tmem_base + C::O_COL + t * HD;
#pragma unroll
        for (int kk = 0; kk < BKV / 16; ++kk)
          umma_bf16_ts_w(leader, d, pa + kk * 8, vd + uint64_t((kk * 2048) >> 4), idesc_o, (j > 0 || kk > 0) ? 1u : 0u);
        umma_commit_w(leader, &s.pv_done[t][j & 1]);
      };
      int ring = 0;
      auto wait_tile = [&](int& stage) {      // next ring entry, in the producer's order
        stage = ring % STAGES;
        const uint32_t phase = (ring / STAGES) & 1;
        ++ring;
        return mbar_wait_relaxed(&s.kv_full[stage], phase);
      };
      bool ok = mbar_wait_relaxed(&s.q_full, 0);
      for (int j = 0; j < 2 && j < n_tiles && ok; ++j) {
        int sk;
        ok = wait_tile(sk);
        if (!ok) break;
        tc_fence_after();
        for (int t = 0; t < NQT; ++t) issue_s(t, j, sk);
        umma_commit_w(leader, &s.kv_empty[sk]);
      }
      for (int jj = 0; jj < n_tiles && ok && !s.abort; ++jj) {
        int sv, sk = 0;
        ok = wait_tile(sv);
        const bool more = jj + 2 < n_tiles;
        for (int t = 0; t < NQT && ok; ++t) {
          ok = mbar_wait_relaxed(&s.p_ready[t][jj & 1], (jj >> 1) & 1);
          if (!ok) break;
          tc_fence_after();
          issue_pv(t, jj, sv);
          if (more) {
            // the scores of key tile jj+2 go into the buffer P_t(jj) occupies: the tensor pipe runs
            // its instructions in order, so the product above has read P before this overwrites it
            if (t == 0) {
              ok = wait_tile(sk);
              if (!ok) break;
              tc_fence_after();
            }
            issue_s(t, jj + 2, sk);
          }
        }
        if (ok) {
          umma_commit_w(leader, &s.kv_empty[sv]);
          if (more) umma_commit_w(leader, &s.kv_empty[sk]);
        }
      }
      if (!ok) POP_ABORT(s, status);
    }
  } else {
    // ------------------------------------------------------------------ softmax warpgroups
    const int t = warp >> 2;                              // query tile of this warpgroup
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;                  // row in the tile == TMEM lane
    const int pos = pos0 + row;                           // absolute query position
    const uint32_t lane_addr = uint32_t(quarter * 32) << 16;
    const uint32_t s_addr = tmem_base + lane_addr + C::S_COL + t * 2 * BKV;
    const uint32_t o_addr = tmem_base + lane_addr + C::O_COL + t * HD;
    float m_run = -INFINITY;      // running (possibly stale) maximum, log2 domain
    float l_run = 0.f;
    bool ok = true;
    // completion of the P V product of key tile j: barrier pv_done[t][j & 1], parity (j >> 1) & 1
    auto wait_pv = [&](int j) { return mbar_wait(&s.pv_done[t][j & 1], (j >> 1) & 1); };

    for (int jj = 0; jj < n_tiles && !s.abort; ++jj) {
      const int kv0 = (j_lo + jj) * BKV;
      const uint32_t sp_addr = s_addr + (jj & 1) * BKV;
      if (!mbar_wait(&s.s_full[t][jj & 1], (jj >> 1) & 1)) { ok = false; break; }
      tc_fence_after();
      float sv[BKV];
#pragma unroll
      for (int c = 0; c < BKV / 32; ++c)
        tmem_ld_32x32b_x32(sp_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[c * 32]));
      tmem_wait_ld();
      // mask (diagonal / window-edge tiles only), then the row maximum of the raw scores on four
      // independent chains of three-input max
      const bool partial = (kv0 + BKV - 1 > pos0) || (p.window > 0 && kv0 <= pos0 + 127 - p.window);
      if (partial) {
        const int lo = p.window > 0 ? pos - p.window : -1;   // valid keys: lo < j <= pos
#pragma unroll
        for (int i = 0; i < BKV; ++i) {
          const int j = kv0 + i;
          if (!(j <= pos && j > lo)) sv[i] = -INFINITY;
        }
      }
      // P = exp2(S * scale - m) with packed fp32 pairs, summed on two chains, rounded to bf16 (key 2c in
      // the low half of packed column c, key 2c+1 in the high half). The exponentials are taken against
      // the maximum the row already has: nothing in them depends on this tile's own maximum, which is
      // reduced alongside (four chains of three-input max) and only checked afterwards.
      float2 acc0, acc1;
      uint32_t pk[BKV / 2];
      float mx0, mx1, mx2, mx3;
      auto exps = [&](float m_use) {
        const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
        const float2 nm2 = make_float2(-m_use, -m_use);
        acc0 = make_float2(0.f, 0.f);
        acc1 = make_float2(0.f, 0.f);
        mx0 = sv[0]; mx1 = sv[2]; mx2 = sv[4]; mx3 = sv[6];
#pragma unroll
        for (int c = 0; c < BKV / 8; ++c) {
          float2 x0 = __ffma2_rn(make_float2(sv[c * 8 + 0], sv[c * 8 + 1]), sc2, nm2);
          float2 x1 = __ffma2_rn(make_float2(sv[c * 8 + 2], sv[c * 8 + 3]), sc2, nm2);
          float2 x2 = __ffma2_rn(make_float2(sv[c * 8 + 4], sv[c * 8 + 5]), sc2, nm2);
          float2 x3 = __ffma2_rn(make_float2(sv[c * 8 + 6], sv[c * 8 + 7]), sc2, nm2);
          mx0 = max3(mx0, sv[c * 8 + 0], sv[c * 8 + 1]);
          mx1 = max3(mx1, sv[c * 8 + 2], sv[c * 8 + 3]);
          mx2 = max3(mx2, sv[c * 8 + 4], sv[c * 8 + 5]);
          mx3 = max3(mx3, sv[c * 8 + 6], sv[c * 8 + 7]);
          x0.x = ex2(x0.x); x0.y = ex2(x0.y);
          x1.x = ex2(x1.x); x1.y = ex2(x1.y);
          x2.x = ex2(x2.x); x2.y = ex2(x2.y);
          x3.x = ex2(x3.x); x3.y = ex2(x3.y);
          acc0 = __fadd2_rn(acc0, x0);
          acc1 = __fadd2_rn(acc1, x1);
          acc0 = __fadd2_rn(acc0, x2);
          acc1 = __fadd2_rn(acc1, x3);
          pk[c * 4 + 0] = pack2(x0.x, x0.y);
          pk[c * 4 + 1] = pack2(x1.x, x1.y);
          pk[c * 4 + 2] = pack2(x2.x, x2.y);
          pk[c * 4 + 3] = pack2(x3.x, x3.y);
        }
      };
      exps(m_run == -INFINITY ? 0.f : m_run);
      const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2;   // log2 domain
      const float m_new = fmaxf(m_run, mx);
      const bool need = (m_new - m_run > 8.0f) || (m_run == -INFINITY && m_new > -INFINITY);
      if (__any_sync(0xffffffffu, need)) {
        // the maximum grew by more than 2^8 somewhere in this warp (in practice: a row's first tiles):
        // rescale the accumulator to the new maximum and take the exponentials again
        const float factor = (m_new == -INFINITY) ? 1.0f : ex2(m_run - m_new);   // ex2(-inf) = 0
        if (jj > 0) {
          if (!wait_pv(jj - 1)) { ok = false; break; }
          tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < HD / 32; ++c) {
            uint32_t o[32];
            tmem_ld_32x32b_x32(o_addr + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
            tmem_st_32x32b_x32(o_addr + c * 32, o);
          }
          tmem_wait_st();
        }
        l_run *= factor;
        m_run = m_new;
        exps(m_run == -INFINITY ? 0.f : m_run);
      }
      l_run += (acc0.x + acc0.y) + (acc1.x + acc1.y);
      tmem_st_32x32b_x32(sp_addr, pk);      // over the scores this thread has just consumed
      tmem_wait_st();
      // cache rows at positions >= kv_len may hold anything: zero them in the staged V tile so that
      // 0 * garbage cannot poison the accumulator (only the last key tile can contain such rows,
      // and its V tile is the last entry of the ring)
      if (kv0 + BKV > kv_len) {
        const int rv = 2 * n_tiles - 1;
        if (!mbar_wait(&s.kv_full[rv % STAGES], (rv / STAGES) & 1)) { ok = false; break; }
        if (t == 0 && row < BKV && kv0 + row >= kv_len) {
          for (int c = 0; c < HD / 64; ++c) {
            uint4* dst = reinterpret_cast<uint4*>(s.kv[rv % STAGES] + c * C::KV_SUB_BYTES + row * 128);
#pragma unroll
            for (int q = 0; q < 8; ++q) dst[q] = make_uint4(0, 0, 0, 0);
          }
        }
        fence_proxy_async_smem();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&s.p_ready[t][jj & 1]);
    }
    if (ok && !s.abort) {
      if (!wait_pv(n_tiles - 1)) {
        ok = false;
      } else {
        tc_fence_after();
        const float inv = 1.0f / l_run;
        const int seq_row = q_row0 + row;
        const bool store = seq_row < seq_len;
        bf16* out = p.out + ((int64_t)row_base + seq_row) * p.ldo + (int64_t)(head0 + t) * HD;
#pragma unroll 1
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t o[32];
          tmem_ld_32x32b_x32(o_addr + c * 32, o);
          tmem_wait_ld();
          if (store) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              uint4 w;
              w.x = pack2(__uint_as_float(o[v * 8 + 0]) * inv, __uint_as_float(o[v * 8 + 1]) * inv);
              w.y = pack2(__uint_as_float(o[v * 8 + 2]) * inv, __uint_as_float(o[v * 8 + 3]) * inv);
              w.z = pack2(__uint_as_float(o[v * 8 + 4]) * inv, __uint_as_float(o[v * 8 + 5]) * inv);
              w.w = pack2(__uint_as_float(o[v * 8 + 6]) * inv, __uint_as_float(o[v * 8 + 7]) * inv);
              *reinterpret_cast<uint4*>(out + c * 32 + v * 8) = w;
            }
          }
        }
      }
    }
    if (!ok) POP_ABORT(s, status);
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (s.abort && threadIdx.x == 0) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);   // let in-flight bulk copies land
  }
  __syncthreads();
  if (warp == NQT * 4 + 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------------
// Variant for head_dim <= 128: the scores of TWO consecutive 64-key tiles are produced by one set of
// 128-wide tensor-core instructions (a 64-wide instruction occupies the pipe as long as a 128-wide
// one), into the two adjacent score buffers of the tile. The softmax and the P V products still
// work on 64 keys at a time, so P V of the first half runs while the second half is in the softmax.
// K and V travel in 128-key stages. The next pair's scores can only be issued once both halves'
// P have been consumed; the other query tile's work fills the tensor pipe in the meantime.
template <int HD, int NQT>
struct PC {
  static constexpr int BKV = 64;                       // softmax / P V granularity
  static constexpr int PKV = 128;                      // keys per stage and per score instruction set
  static constexpr int KV_TILE_BYTES = PKV * HD * 2;
  static constexpr int KV_SUB_BYTES = PKV * 128;       // one 64-wide slice of head_dim
  static constexpr int Q_TILE_BYTES = 128 * HD * 2;
  static constexpr int RING_BYTES = kSmemLimit - 3 * 1024 - NQT * Q_TILE_BYTES;
  static constexpr int STAGES = RING_BYTES / KV_TILE_BYTES < 8 ? RING_BYTES / KV_TILE_BYTES : 8;
  static constexpr int THREADS = NQT * 128 + 64;
  static constexpr int S_COL = 0;                      // S_t[h] at (t * 2 + h) * 64, h = half of the pair
  static constexpr int O_COL = NQT * 2 * BKV;
  static constexpr int COLS_USED = O_COL + NQT * HD;
  static constexpr uint32_t TMEM_COLS = COLS_USED <= 128 ? 128 : (COLS_USED <= 256 ? 256 : 512);
  static_assert(COLS_USED <= 512, "TMEM budget");
  static_assert(STAGES >= 4, "ring too shallow");
};

template <int HD, int NQT>
struct __align__(1024) PairSmem {
  using C = PC<HD, NQT>;
  uint8_t q[NQT][C::Q_TILE_BYTES];
  uint8_t kv[C::STAGES][C::KV_TILE_BYTES];
  uint64_t q_full;
  uint64_t kv_full[C::STAGES];
  uint64_t kv_empty[C::STAGES];
  uint64_t s_full[NQT];         // both halves' scores of a pair complete; phase = pair
  uint64_t p_ready[NQT][2];     // P of half h written over its scores; phase = pair
  uint64_t pv_done[NQT][2];     // O_t += P_t[h] V complete; phase = pair
  uint32_t tmem_base;
  uint32_t raised;
  volatile uint32_t abort;
};

template <int HD, int NQT>
__global__ void __launch_bounds__(PC<HD, NQT>::THREADS, 1)
attn_pair_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const AttnDev p, int* __restrict__ status) {
  using C = PC<HD, NQT>;
  constexpr int BKV = C::BKV, PKV = C::PKV;
  constexpr int STAGES = C::STAGES;
  extern __shared__ uint8_t smem_raw[];
  PairSmem<HD, NQT>& s =
      *reinterpret_cast<PairSmem<HD, NQT>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  const int q_tile = p.q_tiles - 1 - (int)blockIdx.y;    // heaviest query tiles first
  const int head0 = blockIdx.x * NQT;
  const int b = blockIdx.z;
  const int kv_head = head0 * p.n_kv_heads / p.n_q_heads;
  const int q_row0 = q_tile * 128;
  const int row_base = p.cu ? p.cu[b] : b * p.seq_len;   // ragged batches: see attn_kernel
  const int seq_len = p.cu ? p.cu[b + 1] - row_base : p.seq_len;
  const int kv_len = p.cu ? seq_len : p.kv_len;
  if (q_row0 >= seq_len) return;
  const int pos0 = p.q_pos0 + q_row0;
  const int last_pos = min(pos0 + 127, p.q_pos0 + seq_len - 1);
  const int j_hi = min(last_pos, kv_len - 1) / BKV;
  const int j_lo = p.window > 0 ? max(0, pos0 - p.window + 1) / BKV : 0;
  const int n_tiles = j_hi - j_lo + 1;                   // 64-key tiles
  const int n_pairs = (n_tiles + 1) >> 1;

  if (status_raised(status, &s.raised)) return;
  if (threadIdx.x == 0) {
    mbar_init(&s.q_full, 1);
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(&s.kv_full[i], 1);
      mbar_init(&s.kv_empty[i], 1);
    }
    for (int t = 0; t < NQT; ++t) {
      mbar_init(&s.s_full[t], 1);
      for (int i = 0; i < 2; ++i) {
        mbar_init(&s.p_ready[t][i], 4);
        mbar_init(&s.pv_done[t][i], 1);
      }
    }
    s.abort = 0;
    fence_barrier_init();
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
  }
  if (warp == NQT * 4 + 1) {
    tmem_alloc(&s.tmem_base, C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s.tmem_base;

  if (warp == NQT * 4) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(&s.q_full, NQT * C::Q_TILE_BYTES);
      for (int t = 0; t < NQT; ++t)
        for (int c = 0; c < HD / 64; ++c)
          tma_load_3d(s.q[t] + c * 16384, &tmQ, &s.q_full, c * 64, head0 + t, row_base + q_row0);
      const int32_t* bt = p.block_table + (int64_t)b * p.max_pages_per_seq;
      const int loads_per_tile = PKV / p.rows_per_load;
      // ring order: K_0, V_0, K_1, V_1, ... (128-key stages)
      bool ok = true;
      for (int ring = 0; ring < 2 * n_pairs && ok && !s.abort; ++ring) {
        const int J = ring >> 1;
        const CUtensorMap* tm = (ring & 1) ? &tmV : &tmK;
        const int kv0 = (j_lo + 2 * J) * BKV;
        const int stage = ring % STAGES;
        const uint32_t phase = (ring / STAGES) & 1;
        if (!mbar_wait_relaxed(&s.kv_empty[stage], phase ^ 1)) {
          POP_ABORT(s, status);
          ok = false;
          break;
        }
        int n_loads = 0;
        for (int r = 0; r < loads_per_tile; ++r)
          if (kv0 + r * p.rows_per_load < kv_len) ++n_loads;
        mbar_expect_tx(&s.kv_full[stage], n_loads * p.rows_per_load * HD * 2);
        for (int r = 0; r < n_loads; ++r) {
          const int pos = kv0 + r * p.rows_per_load;
          const int page = bt[pos / p.page_size];
          // an entry outside the pool cannot fault here (the tensor map clips), but it is an error
          if ((unsigned)page >= (unsigned)p.num_pages) atomicMin(status, (int)POP_E_INVALID);
          const int slot = pos % p.page_size;
          for (int c = 0; c < HD / 64; ++c)
            tma_load_4d(s.kv[stage] + c * C::KV_SUB_BYTES + r * p.rows_per_load * 128, tm, &s.kv_full[stage],
                        c * 64, kv_head, slot, page);
        }
      }
    }
  } else if (warp == NQT * 4 + 1) {
    // ------------------------------------------------------------------ MMA issuer (whole warp, elected lane)
    const uint32_t leader = elect_one();
    constexpr uint32_t idesc_s = umma_idesc_bf16(128, PKV, 0, 0);
    constexpr uint32_t idesc_o = umma_idesc_bf16(128, HD, 0, 1);
    uint64_t q_desc[NQT];
    for (int t = 0; t < NQT; ++t) q_desc[t] = umma_smem_desc(smem_u32(s.q[t]), 16, 1024);
    const uint64_t k_desc0 = umma_smem_desc(smem_u32(s.kv[0]), 16, 1024);                 // K-major
    const uint64_t v_desc0 = umma_smem_desc(smem_u32(s.kv[0]), C::KV_SUB_BYTES, 1024);    // MN-major
    auto issue_s = [&](int t, int stage) {               // 128 keys -> both score buffers of tile t
      const uint64_t qd = q_desc[t];
      const uint64_t kd = k_desc0 + uint64_t(stage * (C::KV_TILE_BYTES >> 4));
      const uint32_t d = tmem_base + C::S_COL + t * 2 * BKV;
#pragma unroll
      for (int kk = 0; kk < HD / 16; ++kk) {
        const uint64_t ad = qd + uint64_t(((kk >> 2) * 16384 + (kk & 3) * 32) >> 4);
        const uint64_t bd = kd + uint64_t(((kk >> 2) * C::KV_SUB_BYTES + (kk & 3) * 32) >> 4);
        umma_bf16_ss_w(leader, d, ad, bd, idesc_s, kk > 0 ? 1u : 0u);
      }
      umma_commit_w(leader, &s.s_full[t]);
    };
    auto issue_pv = [&](int t, int jj, int stage) {      // 64 keys: half jj & 1 of the pair's V stage
      const int h = jj & 1;
      const uint32_t pa = tmem_base + C::S_COL + (t * 2 + h) * BKV;
      const uint64_t vd = v_desc0 + uint64_t((stage * C::KV_TILE_BYTES + h * BKV * 128) >> 4);
      const uint32_t d = tmem_base + C::O_COL + t * HD;
#pragma unroll
      for (int kk = 0; kk < BKV / 16; ++kk)
        umma_bf16_ts_w(leader, d, pa + kk * 8, vd + uint64_t((kk * 2048) >> 4), idesc_o,
                       (jj > 0 || kk > 0) ? 1u : 0u);
      umma_commit_w(leader, &s.pv_done[t][h]);
    };
    bool ok = mbar_wait_relaxed(&s.q_full, 0);
    if (ok) ok = mbar_wait_relaxed(&s.kv_full[0], 0);
    if (ok) {
      tc_fence_after();
      for (int t = 0; t < NQT; ++t) issue_s(t, 0);
      umma_commit_w(leader, &s.kv_empty[0]);
    }
    for (int J = 0; J < n_pairs && ok && !s.abort; ++J) {
      const int rv = 2 * J + 1, rk = 2 * J + 2;
      const int sv = rv % STAGES, sk = rk % STAGES;
      const bool more = J + 1 < n_pairs;
      ok = mbar_wait_relaxed(&s.kv_full[sv], (rv / STAGES) & 1);
      bool k_ready = false;
      for (int h = 0; h < 2 && ok; ++h) {
        const int jj = 2 * J + h;
        if (jj >= n_tiles) break;
        const bool last_half = (h == 1) || (jj + 1 >= n_tiles);
        for (int t = 0; t < NQT && ok; ++t) {
          ok = mbar_wait_relaxed(&s.p_ready[t][h], J & 1);
          if (!ok) break;
          tc_fence_after();
          issue_pv(t, jj, sv);
          if (last_half && more) {
            // both score buffers of tile t are consumed (the pipe runs in order): next pair's scores
            if (!k_ready) {
              ok = mbar_wait_relaxed(&s.kv_full[sk], (rk / STAGES) & 1);
              if (!ok) break;
              tc_fence_after();
              k_ready = true;
            }
            issue_s(t, sk);
          }
        }
      }
      if (ok) {
        umma_commit_w(leader, &s.kv_empty[sv]);
        if (more) umma_commit_w(leader, &s.kv_empty[sk]);
      }
    }
    if (!ok) POP_ABORT(s, status);
  } else {
    // ------------------------------------------------------------------ softmax warpgroups
    const int t = warp >> 2;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const int pos = pos0 + row;
    const uint32_t lane_addr = uint32_t(quarter * 32) << 16;
    const uint32_t s_addr = tmem_base + lane_addr + C::S_COL + t * 2 * BKV;
    const uint32_t o_addr = tmem_base + lane_addr + C::O_COL + t * HD;
    float m_run = -INFINITY;
    float l_run = 0.f;
    bool ok = true;
    // P V product of 64-key tile j: barrier pv_done[t][j & 1], phase = pair j >> 1
    auto wait_pv = [&](int j) { return mbar_wait(&s.pv_done[t][j & 1], (j >> 1) & 1); };

    for (int jj = 0; jj < n_tiles && !s.abort; ++jj) {
      const int J = jj >> 1, h = jj & 1;
      const int kv0 = (j_lo + jj) * BKV;
      const uint32_t sp_addr = s_addr + h * BKV;
      if (h == 0) {
        if (!mbar_wait(&s.s_full[t], J & 1)) { ok = false; break; }
        tc_fence_after();
      }
      float sv[BKV];
#pragma unroll
      for (int c = 0; c < BKV / 32; ++c)
        tmem_ld_32x32b_x32(sp_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[c * 32]));
      tmem_wait_ld();
      const bool partial = (kv0 + BKV - 1 > pos0) || (p.window > 0 && kv0 <= pos0 + 127 - p.window);
      if (partial) {
        const int lo = p.window > 0 ? pos - p.window : -1;   // valid keys: lo < j <= pos
#pragma unroll
        for (int i = 0; i < BKV; ++i) {
          const int j = kv0 + i;
          if (!(j <= pos && j > lo)) sv[i] = -INFINITY;
        }
      }
      // P = exp2(S * scale - m) with packed fp32 pairs, summed on two chains, rounded to bf16 (key 2c in
      // the low half of packed column c, key 2c+1 in the high half). The exponentials are taken against
      // the maximum the row already has: nothing in them depends on this tile's own maximum, which is
      // reduced alongside (four chains of three-input max) and only checked afterwards.
      float2 acc0, acc1;
      uint32_t pk[BKV / 2];
      float mx0, mx1, mx2, mx3;
      auto exps = [&](float m_use) {
        const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
        const float2 nm2 = make_float2(-m_use, -m_use);
        acc0 = make_float2(0.f, 0.f);
        acc1 = make_float2(0.f, 0.f);
        mx0 = sv[0]; mx1 = sv[2]; mx2 = sv[4]; mx3 = sv[6];
#pragma unroll
        for (int c = 0; c < BKV / 8; ++c) {
          float2 x0 = __ffma2_rn(make_float2(sv[c * 8 + 0], sv[c * 8 + 1]), sc2, nm2);
          float2 x1 = __ffma2_rn(make_float2(sv[c * 8 + 2], sv[c * 8 + 3]), sc2, nm2);
          float2 x2 = __ffma2_rn(make_float2(sv[c * 8 + 4], sv[c * 8 + 5]), sc2, nm2);
          float2 x3 = __ffma2_rn(make_float2(sv[c * 8 + 6], sv[c * 8 + 7]), sc2, nm2);
          mx0 = max3(mx0, sv[c * 8 + 0], sv[c * 8 + 1]);
          mx1 = max3(mx1, sv[c * 8 + 2], sv[c * 8 + 3]);
          mx2 = max3(mx2, sv[c * 8 + 4], sv[c * 8 + 5]);
          mx3 = max3(mx3, sv[c * 8 + 6], sv[c * 8 + 7]);
          x0.x = ex2(x0.x); x0.y = ex2(x0.y);
          x1.x = ex2(x1.x); x1.y = ex2(x1.y);
          x2.x = ex2(x2.x); x2.y = ex2(x2.y);
          x3.x = ex2(x3.x); x3.y = ex2(x3.y);
          acc0 = __fadd2_rn(acc0, x0);
          acc1 = __fadd2_rn(acc1, x1);
          acc0 = __fadd2_rn(acc0, x2);
          acc1 = __fadd2_rn(acc1, x3);
          pk[c * 4 + 0] = pack2(x0.x, x0.y);
          pk[c * 4 + 1] = pack2(x1.x, x1.y);
          pk[c * 4 + 2] = pack2(x2.x, x2.y);
          pk[c * 4 + 3] = pack2(x3.x, x3.y);
        }
      };
      exps(m_run == -INFINITY ? 0.f : m_run);
      const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2;   // log2 domain
      const float m_new = fmaxf(m_run, mx);
      const bool need = (m_new - m_run > 8.0f) || (m_run == -INFINITY && m_new > -INFINITY);
      if (__any_sync(0xffffffffu, need)) {
        // the maximum grew by more than 2^8 somewhere in this warp (in practice: a row's first tiles):
        // rescale the accumulator to the new maximum and take the exponentials again
        const float factor = (m_new == -INFINITY) ? 1.0f : ex2(m_run - m_new);   // ex2(-inf) = 0
        if (jj > 0) {
          if (!wait_pv(jj - 1)) { ok = false; break; }
          tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < HD / 32; ++c) {
            uint32_t o[32];
            tmem_ld_32x32b_x32(o_addr + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
            tmem_st_32x32b_x32(o_addr + c * 32, o);
          }
          tmem_wait_st();
        }
        l_run *= factor;
        m_run = m_new;
        exps(m_run == -INFINITY ? 0.f : m_run);
      }
      l_run += (acc0.x + acc0.y) + (acc1.x + acc1.y);
      tmem_st_32x32b_x32(sp_addr, pk);      // over the scores this thread has just consumed
      tmem_wait_st();
      // cache rows at positions >= kv_len may hold anything: zero them in the pair's staged V tile
      // (128 rows, one per thread of warpgroup 0) before either half's product can read them
      const int pair_kv0 = (j_lo + 2 * J) * BKV;
      if (pair_kv0 + PKV > kv_len) {
        const int rv = 2 * J + 1;
        if (!mbar_wait(&s.kv_full[rv % STAGES], (rv / STAGES) & 1)) { ok = false; break; }
        if (t == 0 && pair_kv0 + row >= kv_len) {
          for (int c = 0; c < HD / 64; ++c) {
            uint4* dst = reinterpret_cast<uint4*>(s.kv[rv % STAGES] + c * C::KV_SUB_BYTES + row * 128);
#pragma unroll
            for (int q = 0; q < 8; ++q) dst[q] = make_uint4(0, 0, 0, 0);
          }
        }
        fence_proxy_async_smem();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&s.p_ready[t][h]);
    }
    if (ok && !s.abort) {
      if (!wait_pv(n_tiles - 1)) {
        ok = false;
      } else {
        tc_fence_after();
        const float inv = 1.0f / l_run;
        const int seq_row = q_row0 + row;
        const bool store = seq_row < seq_len;
        bf16* out = p.out + ((int64_t)row_base + seq_row) * p.ldo + (int64_t)(head0 + t) * HD;
#pragma unroll 1
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t o[32];
          tmem_ld_32x32b_x32(o_addr + c * 32, o);
          tmem_wait_ld();
          if (store) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              uint4 w;
              w.x = pack2(__uint_as_float(o[v * 8 + 0]) * inv, __uint_as_float(o[v * 8 + 1]) * inv);
              w.y = pack2(__uint_as_float(o[v * 8 + 2]) * inv, __uint_as_float(o[v * 8 + 3]) * inv);
              w.z = pack2(__uint_as_float(o[v * 8 + 4]) * inv, __uint_as_float(o[v * 8 + 5]) * inv);
              w.w = pack2(__uint_as_float(o[v * 8 + 6]) * inv, __uint_as_float(o[v * 8 + 7]) * inv);
              *reinterpret_cast<uint4*>(out + c * 32 + v * 8) = w;
            }
          }
        }
      }
    }
    if (!ok) POP_ABORT(s, status);
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (s.abort && threadIdx.x == 0) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);   // let in-flight bulk copies land
  }
  __syncthreads();
  if (warp == NQT * 4 + 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

template <int HD, int NQT, bool PAIR>
int launch_t(const AttnArgs& a, cudaStream_t stream) {
  using C = typename std::conditional<PAIR, PC<HD, NQT>, AC<HD, NQT>>::type;
  AttnDev p;
  p.out = a.out;
  p.ldo = a.ldo;
  p.block_table = a.block_table;
  p.max_pages_per_seq = a.max_pages_per_seq;
  p.page_size = a.page_size;
  p.rows_per_load = a.page_size < C::BKV ? a.page_size : C::BKV;
  p.seq_len = a.seq_len;
  p.q_pos0 = a.q_pos0;
  p.kv_len = a.kv_len;
  p.n_q_heads = a.n_q_heads;
  p.n_kv_heads = a.n_kv_heads;
  p.window = a.window;
  p.num_pages = a.num_pages;
  p.q_tiles = ceil_div(a.seq_len, 128);
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  p.cu = a.cu_seqlens;
  if (C::BKV % p.rows_per_load) return POP_E_INVALID;

  CUtensorMap tq, tk, tv;
  // Q [batch*seq][heads][hd] (row stride ldq)
  {
    const uint64_t rows = a.total_rows > 0 ? (uint64_t)a.total_rows : (uint64_t)a.batch * a.seq_len;
    const uint64_t dims[5] = {(uint64_t)HD, (uint64_t)a.n_q_heads, rows, 1, 1};
    const uint64_t str[4] = {(uint64_t)HD, (uint64_t)a.ldq, (uint64_t)a.ldq * rows, (uint64_t)a.ldq * rows};
    const uint32_t box[5] = {64, 1, 128, 1, 1};
    int rc = make_tmap_bf16_nd(&tq, a.q, 3, dims, str, box);
    if (rc) return rc;
  }
  {
    const uint64_t dims[5] = {(uint64_t)HD, (uint64_t)a.n_kv_heads, (uint64_t)a.page_size, (uint64_t)a.num_pages, 1};
    const uint64_t str[4] = {(uint64_t)HD, (uint64_t)HD * a.n_kv_heads, (uint64_t)HD * a.n_kv_heads * a.page_size,
                             (uint64_t)HD * a.n_kv_heads * a.page_size * a.num_pages};
    const uint32_t box[5] = {64, 1, (uint32_t)p.rows_per_load, 1, 1};
    int rc = make_tmap_bf16_nd(&tk, a.k_pool, 4, dims, str, box);
    if (rc) return rc;
    rc = make_tmap_bf16_nd(&tv, a.v_pool, 4, dims, str, box);
    if (rc) return rc;
  }
  using Smem = typename std::conditional<PAIR, PairSmem<HD, NQT>, AttnSmem<HD, NQT>>::type;
  const size_t smem = sizeof(Smem) + 1024;
  void (*kernel)(CUtensorMap, CUtensorMap, CUtensorMap, AttnDev, int*);
  if constexpr (PAIR) kernel = attn_pair_kernel<HD, NQT>;
  else kernel = attn_kernel<HD, NQT>;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
      return POP_E_CUDA;
    configured = true;
  }
  // CTAs are handed out in blockIdx order, x fastest: all heads of the heaviest query tile first, so the
  // lightest tiles form the tail of the launch
  dim3 grid(a.n_q_heads / NQT, p.q_tiles, a.batch);
  // algorithmic work: 4 * hd flops per unmasked (query, key) pair and query head
  double pairs = 0;
  if (prof_enabled()) {
    for (int r = 0; r < a.seq_len; ++r) {
      const int pos = a.q_pos0 + r;
      pairs += (a.window > 0 && a.window < pos + 1) ? a.window : pos + 1;
    }
  }
  int* status = status_word();
  if (!status) return POP_E_CUDA;
  ProfScope prof(PROF_ATTENTION, 4.0 * HD * pairs * a.n_q_heads * a.batch, stream);
  kernel<<<grid, C::THREADS, smem, stream>>>(tq, tk, tv, p, status);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

}  // namespace

int launch_attention(const AttnArgs& a, cudaStream_t stream) {
  if (!a.q || !a.k_pool || !a.v_pool || !a.block_table || !a.out) return POP_E_INVALID;
  if (a.batch < 1 || a.seq_len < 1 || a.kv_len < 1 || a.n_q_heads < 1 || a.n_kv_heads < 1) return POP_E_INVALID;
  if (a.n_q_heads % a.n_kv_heads || !page_size_ok(a.page_size) || a.ldq % 8 || a.ldo % 8)
    return POP_E_INVALID;
  if (a.q_pos0 + a.seq_len > a.kv_len) return POP_E_INVALID;
  if (a.cu_seqlens != nullptr && (a.q_pos0 != 0 || a.kv_len != a.seq_len)) return POP_E_INVALID;
  if ((int64_t)ceil_div(a.kv_len, a.page_size) > a.max_pages_per_seq) return POP_E_NOSPACE;
  const bool pair = (a.n_q_heads / a.n_kv_heads) % 2 == 0;
  switch (a.head_dim) {
    case 64: return pair ? launch_t<64, 2, true>(a, stream) : launch_t<64, 1, true>(a, stream);
    case 128: return pair ? launch_t<128, 2, true>(a, stream) : launch_t<128, 1, true>(a, stream);
    case 256: return launch_t<256, 1, false>(a, stream);
  }
  return POP_E_INVALID;
}

}  // namespace pop
