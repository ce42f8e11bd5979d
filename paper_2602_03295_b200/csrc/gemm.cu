// bf16 GEMM on the 5th-generation tensor cores: D[M,N] = A[M,K] * B[N,K]^T, fp32 accumulation.
//
// One persistent CTA per SM walks 128 x 256 output tiles. Warp roles:
//   warp 0      TMA producer: streams 128x64 (A) and 256x64 (B) bf16 blocks into a 4-stage
//               shared-memory ring (128-byte swizzle), signalling `full` mbarriers;
//   warp 1      allocates TMEM, issues tcgen05.mma (128x256x16 per instruction) into one of two
//               256-column fp32 accumulators, frees ring stages with tcgen05.commit;
//   warps 2..5  epilogue: tcgen05.ld the finished accumulator (one output row per thread, 32
//               columns at a time), apply the fused epilogue and store, while the MMA warp already
//               fills the other accumulator with the next tile.
// Used for the QKV, O, gate/up and down projections of kept layers (paper Eq. 1-2) and, batched
// over the pruned layers, for their independent K/V projections (Eq. 14).
#include "common.cuh"
#include "ptx.cuh"

#include <cstdlib>

namespace pop {
namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;
constexpr int B_BYTES = BN * BK * 2;
constexpr int GEMM_THREADS = 192;
constexpr int GROUP_M = 16;
constexpr uint32_t TMEM_COLS = 512;
constexpr int OUT_STAGE_BYTES = 32 * 32 * 4;

// Operand ring of the single-CTA form: four stages of a 128 x 64 A block and a 256 x 64 B block, or, with
// 128-column tiles, six stages with a 128 x 64 B block (small problems stream their weights and are bound by
// how many k-blocks a CTA keeps in flight, not by the tensor pipe).
template <int TN>
struct __align__(1024) GemmSmem {
  static constexpr int NST = TN == 128 ? 6 : STAGES;
  static constexpr int TB_BYTES = TN * BK * 2;
  uint8_t a[NST][A_BYTES];
  uint8_t b[NST][TB_BYTES];
  uint8_t out_stage[4][2][OUT_STAGE_BYTES];   // per epilogue warp: two 32-row x 32-float boxes for TMA stores
  uint64_t full[NST];
  uint64_t empty[NST];
  uint64_t tfull[2];
  uint64_t tempty[2];
  uint32_t tmem_base;
  uint32_t raised;
  volatile uint32_t abort;
};

// where the QKV epilogue writes: q rows, and k / v rows into the paged cache
struct RopeEpi {
  bf16* q_out; int64_t ldq;
  bf16* k_pool; bf16* v_pool; int64_t pool_layer_stride;
  int layer0;
  const int32_t* block_table; int max_pages_per_seq; int page_size;
  const float* q_gain; const float* k_gain; int64_t gain_group_stride;
  const float2* table;
  int n_q, n_kv;
  int rows_per_seq, rows_written, pos0;
  float eps;
  const int32_t* cu; int batch; int skip_last;    // ragged batches (see RopeArgs)
  int num_pages;                                  // block-table entries are checked against it when > 0
};

struct GemmDev {
  RopeEpi rope;
  void* out;
  int64_t ldo, out_batch_stride;
  int M, N, K, batch;
  int m_tiles, n_tiles;
  int act, n_valid;
  bf16* hn_out; int64_t ld_hn; const float* gain_next; float* ss_out; int ss_ld;
  const float* ss_in; int ss_cnt; int ss_in_ld; float inv_d; float eps_in;
  const float* a_scale; const float* b_scale;      // FP8 operands: accumulator scale a_scale[row] * *b_scale
  int* status;                                     // device status word
  int group_m;                                     // pair form: 256-row tiles per raster group
};

__device__ __forceinline__ void tile_coords(const GemmDev& p, int t, int& g, int& m, int& n) {
  const int per_batch = p.m_tiles * p.n_tiles;
  g = t / per_batch;
  const int r = t - g * per_batch;
  const int span = GROUP_M * p.n_tiles;
  const int grp = r / span;
  const int first_m = grp * GROUP_M;
  const int gsize = min(GROUP_M, p.m_tiles - first_m);
  const int rr = r - grp * span;
  m = first_m + rr % gsize;
  n = rr / gsize;
}

__device__ __forceinline__ float act_fn(float g, int act) {
  if (act == 0) return g / (1.0f + expf(-g));
  const float c = 0.7978845608028654f;
  return 0.5f * g * (1.0f + tanhf(c * (g + 0.044715f * g * g * g)));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Epilogue of the fused QKV projection (paper Eq. 2-3; Eq. 14 for pruned layers): the thread owns one
// token row of the 128 x TN accumulator tile, which holds TN / HD whole heads (TN = 256, or 128 in the narrow form). q and k heads get
// the optional per-head RMSNorm and RoPE (pair (j, j + HD/2), so two 32-column chunks of TMEM are
// processed together), everything is rounded to bf16; q goes to its row buffer, k and v straight
// into the token's slot of the paged cache. All tcgen05.ld are executed by every lane.
template <int HD, int TN = BN>
__device__ __forceinline__ void qkv_rope_epilogue(const GemmDev& p, uint32_t taddr, int g, int n, int row,
                                                  bool row_ok, float rs) {
  const RopeEpi& r = p.rope;
  constexpr int HALF_CHUNKS = HD / 64;                   // 32-column chunks per half head
  const int total_heads = r.n_q + 2 * r.n_kv;
  int b, i;
  bool active;
  if (r.cu != nullptr) {
    // packed rows: the sequence is the last one starting at or before this row
    int lo = 0, hi = r.batch;                            // cu[lo] <= row < cu[hi] once row < cu[batch]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (r.cu[mid] <= row) lo = mid; else hi = mid;
    }
    b = lo;
    i = row - r.cu[b];
    active = row_ok && row < r.cu[r.batch] && i < r.cu[b + 1] - r.cu[b] - r.skip_last;
  } else {
    b = row / r.rows_per_seq;
    i = row - b * r.rows_per_seq;
    active = row_ok && i < r.rows_written;
  }
  const int pos = r.pos0 + i;
  int64_t cache_row = 0;
  if (active) {
    const int page = r.block_table[(int64_t)b * r.max_pages_per_seq + pos / r.page_size];
    if (r.num_pages > 0 && (unsigned)page >= (unsigned)r.num_pages) {
      atomicMin(p.status, (int)POP_E_INVALID);       // never turned into an address
      active = false;
    } else {
      cache_row = (int64_t)page * r.page_size + pos % r.page_size;
    }
  }
  const float2* tab = r.table + (int64_t)pos * (HD / 2);
#pragma unroll 1
  for (int hh = 0; hh < TN / HD; ++hh) {
    const int head = n * (TN / HD) + hh;
    if (head >= total_heads) break;                      // uniform: depends on the tile only
    const uint32_t haddr = taddr + hh * HD;
    const bool is_q = head < r.n_q;
    const bool is_v = head >= r.n_q + r.n_kv;
    bf16* dst;
    if (is_q) {
      dst = r.q_out + (int64_t)row * r.ldq + (int64_t)head * HD;
    } else {
      const int kvh = is_v ? head - r.n_q - r.n_kv : head - r.n_q;
      bf16* pool = (is_v ? r.v_pool : r.k_pool) + (int64_t)(r.layer0 + g) * r.pool_layer_stride;
      dst = pool + (cache_row * r.n_kv + kvh) * HD;
    }
    if (is_v) {
#pragma unroll 1
      for (int c = 0; c < HD / 32; ++c) {
        uint32_t x[32];
        tmem_ld_32x32b_x32(haddr + c * 32, x);
        tmem_wait_ld();
        if (active) {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
              w[j] = pack_bf16(__uint_as_float(x[v * 8 + j * 2]) * rs, __uint_as_float(x[v * 8 + j * 2 + 1]) * rs);
            *reinterpret_cast<uint4*>(dst + c * 32 + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      continue;
    }
    const float* gain = is_q ? r.q_gain : r.k_gain;
    float rstd = 1.0f;
    if (gain != nullptr) {                               // uniform
      gain += (int64_t)g * r.gain_group_stride;
      float ss = 0.f;
#pragma unroll 1
      for (int c = 0; c < HD / 32; ++c) {
        uint32_t x[32];
        tmem_ld_32x32b_x32(haddr + c * 32, x);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const float t = __uint_as_float(x[e]) * rs;
          ss = fmaf(t, t, ss);
        }
      }
      rstd = rsqrtf(ss / (float)HD + r.eps);
    }
#pragma unroll 1
    for (int c = 0; c < HALF_CHUNKS; ++c) {
      uint32_t lo[32], hi[32];
      tmem_ld_32x32b_x32(haddr + c * 32, lo);
      tmem_ld_32x32b_x32(haddr + (c + HALF_CHUNKS) * 32, hi);
      tmem_wait_ld();
      if (active) {
        float a[32], bq[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const int j = c * 32 + e;
          float x = __uint_as_float(lo[e]) * rs, y = __uint_as_float(hi[e]) * rs;
          if (gain != nullptr) {
            x = x * rstd * gain[j];
            y = y * rstd * gain[j + HD / 2];
          }
          const float2 cs = tab[j];
          a[e] = x * cs.x - y * cs.y;
          bq[e] = y * cs.x + x * cs.y;
        }
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint32_t w[4], z[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            w[j] = pack_bf16(a[v * 8 + j * 2], a[v * 8 + j * 2 + 1]);
            z[j] = pack_bf16(bq[v * 8 + j * 2], bq[v * 8 + j * 2 + 1]);
          }
          *reinterpret_cast<uint4*>(dst + c * 32 + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(dst + HD / 2 + c * 32 + v * 8) = make_uint4(z[0], z[1], z[2], z[3]);
        }
      }
    }
  }
}

// Epilogue of one 128-row x 256-column accumulator slab held in this CTA's TMEM: the calling warp
// (TMEM lane quarter `quarter`) owns rows row0 + quarter*32 .. +31, one row per lane. `n` is the
// 256-column tile index, `boxes` the warp's two 32 x 32 fp32 staging boxes for TMA stores.
// TN: output columns of a tile (256; 128 for the narrow single-CTA form, see launch_gemm)
template <int EPI, int HD, bool FP8, int TN = BN>
__device__ __forceinline__ void epilogue_tile(const GemmDev& p, const CUtensorMap& tmO, uint8_t* boxes,
                                              uint32_t taddr, int g, int row0, int n, int quarter, int lane,
                                              uint32_t& boxes_out) {
  const int row = row0 + quarter * 32 + lane;
  const bool row_ok = row < p.M;
  // rows of a folded RMSNorm arrive un-normalised: their scale comes from the producer's sums
  float rs = 1.0f;
  if (p.ss_in != nullptr && row_ok) {
    float sum = 0.f;
    for (int i = 0; i < p.ss_cnt; ++i) sum += p.ss_in[(int64_t)row * p.ss_in_ld + i];
    rs = rsqrtf(sum * p.inv_d + p.eps_in);
  }
  if (FP8 && row_ok) rs = p.a_scale[row] * *p.b_scale;     // codes -> values: row scale x matrix scale
  if (EPI == EPI_QKV_ROPE) {
    qkv_rope_epilogue<HD == 0 ? 64 : HD, TN>(p, taddr, g, n, row, row_ok, rs);
  } else if (EPI == EPI_GATED_BF16) {
    bf16* out = reinterpret_cast<bf16*>(p.out) + int64_t(g) * p.out_batch_stride + int64_t(row) * p.ldo;
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      uint32_t gr[32], ur[32];
      tmem_ld_32x32b_x32(taddr + c * 32, gr);
      tmem_ld_32x32b_x32(taddr + 128 + c * 32, ur);
      tmem_wait_ld();
      const int col0 = n * 128 + c * 32;
      if (row_ok) {
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          if (col0 + v * 8 + 8 <= p.n_valid) {
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int e = v * 8 + j * 2;
              const float x0 = act_fn(__uint_as_float(gr[e]) * rs, p.act) * (__uint_as_float(ur[e]) * rs);
              const float x1 = act_fn(__uint_as_float(gr[e + 1]) * rs, p.act) * (__uint_as_float(ur[e + 1]) * rs);
              w[j] = pack_bf16(x0, x1);
            }
            *reinterpret_cast<uint4*>(out + col0 + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
  } else if ((EPI == EPI_ADD_F32 || EPI == EPI_STORE_F32) && p.hn_out == nullptr) {
    // fp32 outputs leave through shared memory: the thread writes its 32 values of the chunk as one
    // 128-byte swizzled row of the warp's 32 x 32 box, and an elected lane hands the box to the TMA
    // engine, which stores it or adds it to the residual at the memory side. No residual value
    // is read by the SM, rows and columns beyond the output are clipped by the hardware.
    const bool rows_in = row0 + quarter * 32 < p.M;     // uniform per warp
#pragma unroll 1
    for (int c = 0; c < TN / 32; ++c) {
      if (n * TN + c * 32 >= p.N) break;                 // uniform: the rest of the tile is past the last column
      uint32_t r[32];
      tmem_ld_32x32b_x32(taddr + c * 32, r);
      tmem_wait_ld();
      if (!rows_in) continue;
      // boxes alternate by the count of boxes handed over, so "at most one group still reading"
      // always means the other box
      uint8_t* box = boxes + (boxes_out & 1) * OUT_STAGE_BYTES;
      ++boxes_out;
      if (lane == 0) bulk_wait_read_1();
      __syncwarp();
      uint8_t* mine = box + lane * 128;
#pragma unroll
      for (int v = 0; v < 8; ++v) {
        float4 x = make_float4(__uint_as_float(r[v * 4]), __uint_as_float(r[v * 4 + 1]),
                               __uint_as_float(r[v * 4 + 2]), __uint_as_float(r[v * 4 + 3]));
        if (EPI == EPI_STORE_F32 || FP8) { x.x *= rs; x.y *= rs; x.z *= rs; x.w *= rs; }
        *reinterpret_cast<float4*>(mine + ((v ^ (lane & 7)) << 4)) = x;
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        if (EPI == EPI_ADD_F32) tma_reduce_add_3d(&tmO, box, n * TN + c * 32, row0 + quarter * 32, g);
        else tma_store_3d(&tmO, box, n * TN + c * 32, row0 + quarter * 32, g);
        bulk_commit();
      }
    }
  } else {
    float ss = 0.f;                       // EPI_ADD_F32 with hn_out: sum of squares of this row's new values
#pragma unroll 1
    for (int c = 0; c < TN / 32; ++c) {
      uint32_t r[32];
      tmem_ld_32x32b_x32(taddr + c * 32, r);
      tmem_wait_ld();
      const int col0 = n * TN + c * 32;
      if (row_ok) {
        if (EPI != EPI_ADD_F32) {
#pragma unroll
          for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * rs);
        }
        if (EPI == EPI_STORE_BF16) {
          bf16* out = reinterpret_cast<bf16*>(p.out) + int64_t(g) * p.out_batch_stride + int64_t(row) * p.ldo;
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            if (col0 + v * 8 + 8 <= p.N) {
              uint32_t w[4];
#pragma unroll
              for (int j = 0; j < 4; ++j)
                w[j] = pack_bf16(__uint_as_float(r[v * 8 + j * 2]), __uint_as_float(r[v * 8 + j * 2 + 1]));
              *reinterpret_cast<uint4*>(out + col0 + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        } else {
          float* out = reinterpret_cast<float*>(p.out) + int64_t(g) * p.out_batch_stride + int64_t(row) * p.ldo;
#pragma unroll
          for (int v = 0; v < 8; ++v) {
            if (col0 + v * 4 + 4 <= p.N) {
              float4 x = make_float4(__uint_as_float(r[v * 4]), __uint_as_float(r[v * 4 + 1]),
                                     __uint_as_float(r[v * 4 + 2]), __uint_as_float(r[v * 4 + 3]));
              float4* dst = reinterpret_cast<float4*>(out + col0 + v * 4);
              if (EPI == EPI_ADD_F32) {
                const float4 o = *dst;
                x.x += o.x; x.y += o.y; x.z += o.z; x.w += o.w;
                if (p.hn_out != nullptr) {
                  ss += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
                  const float4 gn = *reinterpret_cast<const float4*>(p.gain_next + col0 + v * 4);
                  uint2 h2;
                  h2.x = pack_bf16(x.x * gn.x, x.y * gn.y);
                  h2.y = pack_bf16(x.z * gn.z, x.w * gn.w);
                  *reinterpret_cast<uint2*>(p.hn_out + (int64_t)row * p.ld_hn + col0 + v * 4) = h2;
                }
              }
              *dst = x;
            }
          }
        }
      }
    }
    if (EPI == EPI_ADD_F32 && p.hn_out != nullptr && row_ok) p.ss_out[(int64_t)row * p.ss_ld + n] = ss;
  }
}

// FP8: the operands are E4M3 codes, a k-block of 128 bytes holds 128 of them (64 bf16 otherwise) and
// one MMA instruction covers 32 (16): the smem tiles, descriptors and their 32-byte steps are the same.
template <int EPI, int HD, bool FP8, int TN = BN>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmO, const GemmDev p,
            int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  using Smem = GemmSmem<TN>;
  constexpr int NST = Smem::NST;
  Smem& s = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int total_tiles = p.m_tiles * p.n_tiles * p.batch;
  constexpr int BKE = FP8 ? 2 * BK : BK;          // operand elements per k-block
  const int k_blocks = (p.K + BKE - 1) / BKE;

  if (status_raised(status, &s.raised)) return;
  if (threadIdx.x == 0) {
    for (int i = 0; i < NST; ++i) {
      mbar_init(&s.full[i], 1);
      mbar_init(&s.empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s.tfull[i], 1);
      mbar_init(&s.tempty[i], 4);
    }
    s.abort = 0;
    fence_barrier_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    tmem_alloc(&s.tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s.tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      for (int t = blockIdx.x; t < total_tiles && !s.abort; t += gridDim.x) {
        int g, m, n;
        tile_coords(p, t, g, m, n);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(&s.empty[stage], phase ^ 1)) {
            s.abort = 1;
            atomicMin(status, (int)POP_E_DEVICE_TIMEOUT);
            break;
          }
          mbar_expect_tx(&s.full[stage], A_BYTES + TN * BK * 2);
          tma_load_3d(s.a[stage], &tmA, &s.full[stage], kb * BKE, m * BM, g);
          tma_load_3d(s.b[stage], &tmB, &s.full[stage], kb * BKE, n * TN, g);
          if (++stage == NST) {
            stage = 0;
            phase ^= 1;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp walks this role with identical values; one elected lane issues.
    {
      const uint32_t leader = elect_one();
      constexpr uint32_t idesc = FP8 ? umma_idesc_e4m3(BM, TN) : umma_idesc_bf16(BM, TN, 0, 0);
      const uint64_t a_desc0 = umma_smem_desc(smem_u32(s.a[0]), 16, 1024);
      const uint64_t b_desc0 = umma_smem_desc(smem_u32(s.b[0]), 16, 1024);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      for (int t = blockIdx.x; t < total_tiles && !s.abort; t += gridDim.x, ++it) {
        const int buf = it & 1;
        const uint32_t bphase = (it >> 1) & 1;
        if (!mbar_wait(&s.tempty[buf], bphase ^ 1)) {
          s.abort = 1;
          atomicMin(status, (int)POP_E_DEVICE_TIMEOUT);
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * TN;
        bool ok = true;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(&s.full[stage], phase)) {
            ok = false;
            break;
          }
          tc_fence_after();
          // only the 16-byte-granular start address in the descriptor's low bits moves
          const uint64_t ad0 = a_desc0 + uint64_t(stage * (A_BYTES >> 4));
          const uint64_t bd0 = b_desc0 + uint64_t(stage * (Smem::TB_BYTES >> 4));
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            if constexpr (FP8)
              umma_e4m3_ss_w(leader, d_tmem, ad0 + uint64_t(k * 2), bd0 + uint64_t(k * 2), idesc,
                             (kb | k) != 0 ? 1u : 0u);
            else
              umma_bf16_ss_w(leader, d_tmem, ad0 + uint64_t(k * 2), bd0 + uint64_t(k * 2), idesc,
                             (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit_w(leader, &s.empty[stage]);
          if (++stage == NST) {
            stage = 0;
            phase ^= 1;
          }
        }
        if (!ok) {
          s.abort = 1;
          atomicMin(status, (int)POP_E_DEVICE_TIMEOUT);
          break;
        }
        umma_commit_w(leader, &s.tfull[buf]);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (4 warps)
    const int quarter = warp & 3;              // TMEM lane quarter this warp may read
    int it = 0;
    uint32_t boxes_out = 0;                     // output boxes this warp has handed to the TMA engine
    for (int t = blockIdx.x; t < total_tiles && !s.abort; t += gridDim.x, ++it) {
      const int buf = it & 1;
      const uint32_t bphase = (it >> 1) & 1;
      int g, m, n;
      tile_coords(p, t, g, m, n);
      if (!mbar_wait(&s.tfull[buf], bphase)) {
        s.abort = 1;
        atomicMin(status, (int)POP_E_DEVICE_TIMEOUT);
        break;
      }
      tc_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + buf * TN;
      epilogue_tile<EPI, HD, FP8, TN>(p, tmO, s.out_stage[quarter][0], taddr, g, m * BM, n, quarter, lane, boxes_out);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&s.tempty[buf]);
    }
  }

  // ------------------------------------------------------------------ teardown
  if (warp >= 2 && lane == 0) bulk_wait_all();   // this lane's output boxes have landed
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (s.abort && threadIdx.x == 0) {
    // give bulk copies that may still be in flight into this CTA's shared memory time to land
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------------
// CTA-pair form for large problems: two CTAs of a cluster (one SM pair) own one 256 x 256 output
// tile. Each CTA streams its own 128 rows of A and its own 128 rows of B (half of the tile's
// columns) into its own shared memory -- 32 KB per k-block instead of 48 KB, six stages instead of
// four -- and the even-ranked CTA issues tcgen05.mma.cta_group::2 (256 x 256 x 16), which reads both
// CTAs' operand halves and leaves each CTA its own 128 x 256 slab of the accumulator in its own
// TMEM. Per output element every SM fetches a third fewer operand bytes from L2 and shared memory.
// No load is multicast; only mbarrier arrivals cross between the two CTAs:
//   full[s]    lives in the even CTA: its producer arms it with the bytes of BOTH CTAs' loads and both
//              CTAs' loads complete their bytes on it;
//   empty[s], tfull[b]   one per CTA, signalled in both CTAs by a multicast tcgen05.commit;
//   tempty[b]  lives in the even CTA, counts the eight epilogue warps of both CTAs.
constexpr int PSTAGES = 6;
constexpr int PB_BYTES = 128 * BK * 2;      // this CTA's half of the B block

struct __align__(1024) PairGemmSmem {
  uint8_t a[PSTAGES][A_BYTES];
  uint8_t b[PSTAGES][PB_BYTES];
  uint8_t out_stage[4][2][OUT_STAGE_BYTES];
  uint64_t full[PSTAGES];
  uint64_t empty[PSTAGES];
  uint64_t tfull[2];
  uint64_t tempty[2];
  uint32_t tmem_base;
  uint32_t raised;
  volatile uint32_t abort;
};

// Raster of the pair form: groups of group_m tile rows; inside a group the tile rows vary fastest, so
// the CTA pairs working at any one time share a few B column panels and the group's A panel, which
// stays in L2 while the group sweeps over all column tiles.
__device__ __forceinline__ void pair_tile_coords(const GemmDev& p, int m_tiles2, int t, int& g, int& m, int& n) {
  const int per_batch = m_tiles2 * p.n_tiles;
  g = t / per_batch;
  const int r = t - g * per_batch;
  const int span = p.group_m * p.n_tiles;
  const int grp = r / span;
  const int first_m = grp * p.group_m;
  const int gsize = min(p.group_m, m_tiles2 - first_m);
  const int rr = r - grp * span;
  m = first_m + rr % gsize;
  n = rr / gsize;
}

template <int EPI, int HD, bool FP8>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmO, const GemmDev p, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  PairGemmSmem& s =
      *reinterpret_cast<PairGemmSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0: issues the tensor-core instructions
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int m_tiles2 = (p.M + 2 * BM - 1) / (2 * BM);
  const int total_tiles = m_tiles2 * p.n_tiles * p.batch;
  constexpr int BKE = FP8 ? 2 * BK : BK;
  const int k_blocks = (p.K + BKE - 1) / BKE;

  // The even CTA decides for the pair whether the status word is raised (a kernel of this library
  // does nothing then), so that both CTAs take the same path through the collective steps below.
  cluster_arrive();      // both CTAs are running: the peer's shared memory may be written from here on
  cluster_wait();
  if (threadIdx.x == 0) {
    s.abort = 0;
    if (rank == 0) {
      const uint32_t v = (*reinterpret_cast<const volatile int*>(status) != 0) ? 1u : 0u;
      s.raised = v;
      st_cluster_u32(mapa_u32(smem_u32(&s.raised), 1), v);
    }
  }
  cluster_arrive();
  cluster_wait();
  if (*reinterpret_cast<volatile uint32_t*>(&s.raised) != 0) return;
  if (threadIdx.x == 0) {
    for (int i = 0; i < PSTAGES; ++i) {
      mbar_init(&s.full[i], 1);        // used in the even CTA, armed by its producer for both CTAs' bytes
      mbar_init(&s.empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s.tfull[i], 1);
      mbar_init(&s.tempty[i], 8);      // used in the even CTA: four epilogue warps of each CTA
    }
    fence_barrier_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    tmem_alloc_pair(&s.tmem_base, TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  // the peer's barriers must exist before anything is signalled across
  cluster_arrive();
  cluster_wait();
  tc_fence_after();
  const uint32_t tmem_base = s.tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      for (int t = pair; t < total_tiles && !s.abort; t += n_pairs) {
        int g, m, n;
        pair_tile_coords(p, m_tiles2, t, g, m, n);
        const int row0 = m * 2 * BM + (int)rank * BM;       // this CTA's rows of A
        const int col0 = n * BN + (int)rank * 128;          // this CTA's rows of B (output columns)
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(&s.empty[stage], phase ^ 1)) {
            s.abort = 1;
            atomicMin(status, (int)POP_E_DEVICE_TIMEOUT);
            break;
          }
          const uint32_t full0 = mapa_u32(smem_u32(&s.full[stage]), 0);
          // The even CTA's one arrival arms the barrier with the bytes of both CTAs' loads; the odd CTA
          // only sends its bytes there. Its loads for this phase cannot start before the phase opens:
          // its empty[stage] fires when the tensor core has finished reading the previous contents,
          // which is after the previous phase completed. Bytes that land before the arming arrival
          // are accounted for when it comes (the pending arrival keeps the phase open).
          if (rank == 0) mbar_expect_tx(&s.full[stage], 2 * (A_BYTES + PB_BYTES));
          tma_load_3d_pair(s.a[stage], &tmA, full0, kb * BKE, row0, g);
          tma_load_3d_pair(s.b[stage], &tmB, full0, kb * BKE, col0, g);
          if (++stage == PSTAGES) {
            stage = 0;
            phase ^= 1;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (even CTA only)
    if (rank == 0) {
      const uint32_t leader = elect_one();
      constexpr uint32_t idesc = FP8 ? umma_idesc_e4m3(2 * BM, BN) : umma_idesc_bf16(2 * BM, BN, 0, 0);
      const uint64_t a_desc0 = umma_smem_desc(smem_u32(s.a[0]), 16, 1024);
      const uint64_t b_desc0 = umma_smem_desc(smem_u32(s.b[0]), 16, 1024);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      for (int t = pair; t < total_tiles && !s.abort; t += n_pairs, ++it) {
        const int buf = it & 1;
        const uint32_t bphase = (it >> 1) & 1;
        if (!mbar_wait(&s.tempty[buf], bphase ^ 1)) {
          s.abort = 1;
          atomicMin(status, (int)POP_E_DEVICE_TIMEOUT);
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN;
        bool ok = true;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(&s.full[stage], phase)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint64_t ad0 = a_desc0 + uint64_t(stage * (A_BYTES >> 4));
          const uint64_t bd0 = b_desc0 + uint64_t(stage * (PB_BYTES >> 4));
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            if constexpr (FP8)
              umma_e4m3_ss_pair_w(leader, d_tmem, ad0 + uint64_t(k * 2), bd0 + uint64_t(k * 2), idesc,
                                  (kb | k) != 0 ? 1u : 0u);
            else
              umma_bf16_ss_pair_w(leader, d_tmem, ad0 + uint64_t(k * 2), bd0 + uint64_t(k * 2), idesc,
                                  (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit_pair_w(leader, &s.empty[stage], (uint16_t)3);      // the stage is free in both CTAs
          if (++stage == PSTAGES) {
            stage = 0;
            phase ^= 1;
          }
        }
        if (!ok) {
          s.abort = 1;
          atomicMin(status, (int)POP_E_DEVICE_TIMEOUT);
          break;
        }
        umma_commit_pair_w(leader, &s.tfull[buf], (uint16_t)3);           // both CTAs' slabs are complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (4 warps per CTA)
    const int quarter = warp & 3;
    int it = 0;
    uint32_t boxes_out = 0;
    for (int t = pair; t < total_tiles && !s.abort; t += n_pairs, ++it) {
      const int buf = it & 1;
      const uint32_t bphase = (it >> 1) & 1;
      int g, m, n;
      pair_tile_coords(p, m_tiles2, t, g, m, n);
      if (!mbar_wait(&s.tfull[buf], bphase)) {
        s.abort = 1;
        atomicMin(status, (int)POP_E_DEVICE_TIMEOUT);
        break;
      }
      tc_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + buf * BN;
      epilogue_tile<EPI, HD, FP8>(p, tmO, s.out_stage[quarter][0], taddr, g, m * 2 * BM + (int)rank * BM, n, quarter,
                                  lane, boxes_out);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_u32(smem_u32(&s.tempty[buf]), 0));
    }
  }

  // ------------------------------------------------------------------ teardown
  if (warp >= 2 && lane == 0) bulk_wait_all();
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (s.abort && threadIdx.x == 0) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);   // let copies still in flight into this CTA land
  }
  // neither CTA may release its TMEM or exit while the other can still signal it or read its operands
  cluster_arrive();
  cluster_wait();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

template <int EPI, int HD = 0, bool FP8 = false>
int launch_epi(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& to, const GemmDev& p_in, int grid,
               bool pair, bool narrow, cudaStream_t stream) {
  int* status = status_word();
  if (!status) return POP_E_CUDA;
  GemmDev p = p_in;
  p.status = status;
  if (pair) {
    const size_t smem = sizeof(PairGemmSmem) + 1024;
    static bool configured = false;
    if (!configured) {
      if (cudaFuncSetAttribute(gemm_pair_kernel<EPI, HD, FP8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)smem) != cudaSuccess)
        return POP_E_CUDA;
      configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(GEMM_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    ProfScope prof(PROF_GEMM, 2.0 * p.M * p.N * p.K * p.batch, stream);
    const cudaError_t e = cudaLaunchKernelEx(&cfg, gemm_pair_kernel<EPI, HD, FP8>, ta, tb, to, p, status);
    count_launch();
    return (e == cudaSuccess && cudaGetLastError() == cudaSuccess) ? POP_OK : POP_E_CUDA;
  }
  const size_t smem = sizeof(GemmSmem<BN>) + 1024;
  if constexpr (EPI == EPI_STORE_BF16 || EPI == EPI_STORE_F32 || EPI == EPI_ADD_F32 ||
                (EPI == EPI_QKV_ROPE && HD >= 64 && HD <= 128)) {
    if (narrow) {
      static bool configured_narrow = false;
      const size_t smem_n = sizeof(GemmSmem<128>) + 1024;
      if (!configured_narrow) {
        if (cudaFuncSetAttribute(gemm_kernel<EPI, HD, FP8, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem_n) != cudaSuccess)
          return POP_E_CUDA;
        configured_narrow = true;
      }
      ProfScope prof(PROF_GEMM, 2.0 * p.M * p.N * p.K * p.batch, stream);
      gemm_kernel<EPI, HD, FP8, 128><<<grid, GEMM_THREADS, smem_n, stream>>>(ta, tb, to, p, status);
      count_launch();
      return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
    }
  }
  if (narrow) return POP_E_INVALID;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(gemm_kernel<EPI, HD, FP8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
      return POP_E_CUDA;
    configured = true;
  }
  ProfScope prof(PROF_GEMM, 2.0 * p.M * p.N * p.K * p.batch, stream);
  gemm_kernel<EPI, HD, FP8><<<grid, GEMM_THREADS, smem, stream>>>(ta, tb, to, p, status);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? POP_OK : POP_E_CUDA;
}

// CTA pairs pay off once every SM pair has at least one 256 x 256 tile; POP_GEMM_PAIR=0 / 1 in the
// environment forces the single-CTA / the pair form (used by the tests to cover both on every shape).
// Tile rows per raster group of the pair form. POP_GEMM_GROUP_M overrides (measurements).
int pair_group_m(int K) {
  const char* e = std::getenv("POP_GEMM_GROUP_M");
  if (e && atoi(e) > 0) return atoi(e);
  (void)K;
  return 16;
}

// Narrow single-CTA form: 128 x 128 tiles for the plain-store, residual and (head_dim <= 128) QKV epilogues when 128 x 256
// tiles would leave at least half of the SMs without a tile (short prompts: the O and down projections of
// 512 rows are 64 tiles). POP_GEMM_NARROW=0 / 1 forces it off / on wherever it is possible.
bool use_narrow(bool possible, int64_t tiles, int sms) {
  if (!possible) return false;
  const char* e = std::getenv("POP_GEMM_NARROW");
  if (e && e[0] == '0') return false;
  if (e && e[0] == '1') return true;
  return tiles * 2 <= sms;      // twice as many narrow tiles are still one wave (B 8 x 32 tokens: -4.6 % per prefill)
}

bool use_pair(int M, int64_t tiles2, int sms) {
  const char* e = std::getenv("POP_GEMM_PAIR");
  if (e && e[0] == '0') return false;
  if (e && e[0] == '1') return true;
  return M > BM && tiles2 >= sms / 2;
}

}  // namespace

int launch_gemm(const GemmArgs& a, cudaStream_t stream) {
  if (!a.A || !a.B || (!a.out && a.epilogue != EPI_QKV_ROPE) || a.M < 1 || a.N < 1 || a.K < 1 || a.batch < 1) return POP_E_INVALID;
  if (a.K % 8 || a.lda % 8 || a.ldb % 8 || a.a_batch_stride % 8 || a.b_batch_stride % 8) return POP_E_INVALID;
  if ((reinterpret_cast<uintptr_t>(a.A) | reinterpret_cast<uintptr_t>(a.B) | reinterpret_cast<uintptr_t>(a.out)) & 15)
    return POP_E_INVALID;
  if (a.epilogue == EPI_QKV_ROPE) {
    const RopeArgs* r = a.rope;
    if (!r || !r->k_pool || !r->v_pool || !r->block_table || !r->table || (r->n_q > 0 && !r->q_out))
      return POP_E_INVALID;
    if ((r->hd != 64 && r->hd != 128 && r->hd != 256) || a.N != (r->n_q + 2 * r->n_kv) * r->hd) return POP_E_INVALID;
    if (r->ldq % 8) return POP_E_INVALID;
    if (r->cu_seqlens == nullptr && (r->rows_per_seq < 1 || a.M % r->rows_per_seq)) return POP_E_INVALID;
    if (r->cu_seqlens != nullptr && (r->batch < 1 || r->skip_last < 0)) return POP_E_INVALID;
  } else if (a.epilogue == EPI_GATED_BF16) {
    if (a.N % 256 || a.n_valid % 8 || a.n_valid > a.N / 2 || a.ldo % 8) return POP_E_INVALID;
  } else if (a.epilogue == EPI_STORE_BF16) {
    if (a.N % 8 || a.ldo % 8) return POP_E_INVALID;
  } else {
    if (a.N % 4 || a.ldo % 4) return POP_E_INVALID;
  }
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return POP_E_CUDA;
  const int64_t tiles2 = int64_t(ceil_div(a.M, 2 * BM)) * ceil_div(a.N, BN) * a.batch;
  const bool pair = use_pair(a.M, tiles2, sms);
  const bool narrow = use_narrow(!pair && a.N > 128 && !a.hn_out && !a.ss_out &&
                                     (a.epilogue == EPI_STORE_BF16 || a.epilogue == EPI_STORE_F32 ||
                                      a.epilogue == EPI_ADD_F32 ||
                                      (a.epilogue == EPI_QKV_ROPE && a.rope && a.rope->hd <= 128)),
                                 int64_t(ceil_div(a.M, BM)) * ceil_div(a.N, BN) * a.batch, sms);
  const uint32_t b_box = (pair || narrow) ? 128 : BN;   // a CTA of a pair loads its own half of the B block
  CUtensorMap ta, tb;
  int rc;
  if (a.fp8) {
    if (a.batch != 1 || !a.a_scale || !a.b_scale || a.K % 16 || a.lda % 16 || a.ldb % 16 || a.hn_out || a.ss_in)
      return POP_E_INVALID;
    rc = make_tmap_u8_3d(&ta, a.A, a.K, a.M, 1, a.lda, (uint64_t)a.lda * a.M, BM);
    if (rc) return rc;
    rc = make_tmap_u8_3d(&tb, a.B, a.K, a.N, 1, a.ldb, (uint64_t)a.ldb * a.N, b_box);
    if (rc) return rc;
  } else {
    rc = make_tmap_bf16_3d(&ta, a.A, a.K, a.M, a.batch, a.lda, a.a_batch_stride ? a.a_batch_stride : a.lda * a.M,
                           BK, BM);
    if (rc) return rc;
    rc = make_tmap_bf16_3d(&tb, a.B, a.K, a.N, a.batch, a.ldb, a.b_batch_stride ? a.b_batch_stride : a.ldb * a.N, BK,
                           b_box);
    if (rc) return rc;
  }
  if (a.hn_out != nullptr) {
    if (a.epilogue != EPI_ADD_F32 || a.batch != 1 || !a.gain_next || !a.ss_out || a.ld_hn % 4 ||
        a.ss_ld < ceil_div(a.N, BN))
      return POP_E_INVALID;
  }
  if (a.ss_in != nullptr && (a.batch != 1 || a.ss_cnt < 1 || a.ss_in_ld < a.ss_cnt || a.norm_d < 1))
    return POP_E_INVALID;
  CUtensorMap to = ta;   // only the fp32 epilogues use it
  if ((a.epilogue == EPI_STORE_F32 || a.epilogue == EPI_ADD_F32) && a.hn_out == nullptr) {
    rc = make_tmap_f32_3d(&to, a.out, a.N, a.M, a.batch, a.ldo,
                          a.out_batch_stride ? a.out_batch_stride : a.ldo * (int64_t)a.M, 32);
    if (rc) return rc;
  }
  GemmDev p{};
  p.hn_out = a.hn_out; p.ld_hn = a.ld_hn; p.gain_next = a.gain_next; p.ss_out = a.ss_out; p.ss_ld = a.ss_ld;
  p.ss_in = a.ss_in; p.ss_cnt = a.ss_cnt; p.ss_in_ld = a.ss_in_ld;
  p.inv_d = a.norm_d > 0 ? 1.0f / (float)a.norm_d : 0.f;
  p.eps_in = a.norm_eps;
  p.a_scale = a.a_scale; p.b_scale = a.b_scale;
  if (a.epilogue == EPI_QKV_ROPE) {
    const RopeArgs& r = *a.rope;
    p.rope.q_out = r.q_out; p.rope.ldq = r.ldq;
    p.rope.k_pool = r.k_pool; p.rope.v_pool = r.v_pool; p.rope.pool_layer_stride = r.pool_layer_stride;
    p.rope.layer0 = r.layer0;
    p.rope.block_table = r.block_table; p.rope.max_pages_per_seq = r.max_pages_per_seq;
    p.rope.page_size = r.page_size;
    p.rope.q_gain = r.q_gain; p.rope.k_gain = r.k_gain; p.rope.gain_group_stride = r.gain_group_stride;
    p.rope.table = r.table;
    p.rope.n_q = r.n_q; p.rope.n_kv = r.n_kv;
    p.rope.rows_per_seq = r.rows_per_seq; p.rope.rows_written = r.rows_written; p.rope.pos0 = r.pos0;
    p.rope.eps = r.eps;
    p.rope.cu = r.cu_seqlens; p.rope.batch = r.batch; p.rope.skip_last = r.skip_last;
    p.rope.num_pages = r.num_pages;
  }
  p.out = a.out;
  p.ldo = a.ldo;
  p.out_batch_stride = a.out_batch_stride;
  p.M = a.M; p.N = a.N; p.K = a.K; p.batch = a.batch;
  p.m_tiles = ceil_div(a.M, BM);
  p.n_tiles = ceil_div(a.N, narrow ? 128 : BN);
  p.act = a.act;
  p.n_valid = a.n_valid;
  const int64_t total = int64_t(p.m_tiles) * p.n_tiles * p.batch;
  int grid = (int)(total < sms ? total : sms);
  if (pair) grid = 2 * (int)(tiles2 < sms / 2 ? tiles2 : sms / 2);
  p.group_m = pair_group_m(a.K);
  if (a.fp8) {
    switch (a.epilogue) {
      case EPI_STORE_BF16: return launch_epi<EPI_STORE_BF16, 0, true>(ta, tb, to, p, grid, pair, narrow, stream);
      case EPI_STORE_F32: return launch_epi<EPI_STORE_F32, 0, true>(ta, tb, to, p, grid, pair, narrow, stream);
      case EPI_ADD_F32: return launch_epi<EPI_ADD_F32, 0, true>(ta, tb, to, p, grid, pair, narrow, stream);
      case EPI_GATED_BF16: return launch_epi<EPI_GATED_BF16, 0, true>(ta, tb, to, p, grid, pair, narrow, stream);
      case EPI_QKV_ROPE:
        switch (a.rope->hd) {
          case 64: return launch_epi<EPI_QKV_ROPE, 64, true>(ta, tb, to, p, grid, pair, narrow, stream);
          case 128: return launch_epi<EPI_QKV_ROPE, 128, true>(ta, tb, to, p, grid, pair, narrow, stream);
          case 256: return launch_epi<EPI_QKV_ROPE, 256, true>(ta, tb, to, p, grid, pair, narrow, stream);
        }
        return POP_E_INVALID;
    }
    return POP_E_INVALID;
  }
  switch (a.epilogue) {
    case EPI_STORE_BF16: return launch_epi<EPI_STORE_BF16>(ta, tb, to, p, grid, pair, narrow, stream);
    case EPI_STORE_F32: return launch_epi<EPI_STORE_F32>(ta, tb, to, p, grid, pair, narrow, stream);
    case EPI_ADD_F32: return launch_epi<EPI_ADD_F32>(ta, tb, to, p, grid, pair, narrow, stream);
    case EPI_GATED_BF16: return launch_epi<EPI_GATED_BF16>(ta, tb, to, p, grid, pair, narrow, stream);
    case EPI_QKV_ROPE:
      switch (a.rope->hd) {
        case 64: return launch_epi<EPI_QKV_ROPE, 64>(ta, tb, to, p, grid, pair, narrow, stream);
        case 128: return launch_epi<EPI_QKV_ROPE, 128>(ta, tb, to, p, grid, pair, narrow, stream);
        case 256: return launch_epi<EPI_QKV_ROPE, 256>(ta, tb, to, p, grid, pair, narrow, stream);
      }
      return POP_E_INVALID;
  }
  return POP_E_INVALID;
}

}  // namespace pop
