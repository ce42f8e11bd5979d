// One position of one sequence through a run of decoder layers as a single cooperative kernel
// (paper Sec. 3.3: the boundary token passes the pruned layers as a decode step; Sec. 3.2, Eq. 11:
// the decode stage uses every layer). The step is bound by the weight stream, so the kernel is built
// around keeping that stream busy: one CTA per SM; in each CTA one producer warp walks the CTA's
// share of every weight matrix and of the cached keys and values of all the layers, in the order
// they are needed, and copies it tile by tile into a ring of shared-memory stages with bulk
// asynchronous copies (cp.async.bulk + mbarrier); eight consumer warps take the tiles. The producer
// never waits for a layer boundary: weights and old cache rows do not depend on the activations, so
// the copies of the next phase are in flight while the consumers are still at the grid-wide barrier
// that separates two phases. Phases of a layer (a grid-wide barrier after each):
//   1  h = bf16(RMSNorm(x)); rows of [W^Q; W^K; W^V] h                          -> qkv (fp32)
//   2  per-head norm (if any), RoPE, cache append, attention over the cache     -> o (bf16)
//   3  x += W^O o
//   4  h = bf16(RMSNorm(x)); a = act(W^gate h) * (W^up h)                        -> a (bf16)
//   5  x += W^down a
// Every output row of a matrix-vector phase belongs to one CTA (rows are dealt out evenly, so no
// sum crosses CTAs); inside a CTA the eight consumer warps split K, and their partial sums meet in
// shared memory in a fixed order. Attention: CTA (kv head, split) covers a contiguous range of cached
// positions with the warp-level tensor-core path (keys on the M side, as in dec_attn_kernel); the new
// position's key and value never go through memory on their way to the scores. The last CTA of a
// kv head to finish merges the splits.
// Every wait (mbarrier, grid barrier) is bounded; a wait that runs out raises the status word and
// an abort flag that makes the other CTAs leave too.
#include "common.cuh"
#include "ptx.cuh"

#include <cstdlib>

namespace pop {
namespace {

constexpr int FW = 8;                              // consumer warps
constexpr int F_THREADS = (FW + 1) * 32;           // + the producer warp
constexpr int F_HD = 128;
constexpr int F_KEYS = 64;                         // cache positions per attention tile
constexpr int F_PITCH = 2 * F_HD + 16;             // bytes between two rows of a K or V tile: 8 rows of a
                                                   // matrix load fall into 8 different 16-byte bank groups
constexpr int F_STAGE = 2 * F_KEYS * F_PITCH;      // K rows, then V rows (34816 B)
constexpr int F_NS = 6;
constexpr int F_MAXJ = 8;                          // 256-element K steps per warp: K <= 8 * 8 * 256
constexpr int F_RT = 8;                            // most weight rows in one tile
constexpr int F_SCRATCH = 16768;
constexpr int F_MAXACC = F_SCRATCH / (FW * 4);     // accumulator rows of one CTA in one phase
constexpr int F_MAXG = 8;                          // query heads per kv head
constexpr int F_SMEM = F_NS * F_STAGE + F_SCRATCH + 256;
constexpr long long F_WAIT_CYCLES = 1000000000ll;  // about half a second
constexpr uint32_t FULLMASK = 0xffffffffu;

typedef FusedDecodeArgs FusedDev;

__device__ __forceinline__ float f_warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULLMASK, v, o);
  return v;
}
__device__ __forceinline__ float bf16_round(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }
__device__ __forceinline__ void f_unpack8(const uint4& raw, float (&f)[8]) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}
__device__ __forceinline__ float f_act(float g, int act) {
  if (act == 0) return g / (1.0f + expf(-g));
  const float c = 0.7978845608028654f;
  return 0.5f * g * (1.0f + tanhf(c * (g + 0.044715f * g * g * g)));
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// barrier of the consumer warps with an OR over `flag`: every thread gets the same answer
__device__ __forceinline__ bool consumer_bar_or(bool flag) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "barrier.red.or.pred p, 1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"(flag ? 1u : 0u), "n"(FW * 32)
      : "memory");
  return r != 0;
}
__device__ __forceinline__ void f_ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void f_ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ uint32_t f_movm_t(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
  return y;
}
__device__ __forceinline__ void f_mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t f_pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// Bounded mbarrier wait that also gives up when the CTA's abort flag is up.
__device__ __forceinline__ bool f_wait(uint64_t* bar, uint32_t parity, const volatile int* s_abort) {
#pragma unroll 1
  for (int i = 0; i < 2048; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i) {
      if (mbar_try_wait(bar, parity)) return true;
      __nanosleep(32);
    }
    if (*s_abort) return false;
    if (clock64() - t0 > F_WAIT_CYCLES) return false;
  }
}

__device__ __forceinline__ void f_fail(const FusedDev& p, volatile int* s_abort) {
  atomicMin(p.status, (int)POP_E_DEVICE_TIMEOUT);
  atomicExch(p.sync + 1, 1u);
  *s_abort = 1;
}

// ------------------------------------------------------------------------------ the CTA's share of a phase
enum { PH_QKV = 0, PH_ATT = 1, PH_O = 2, PH_GU = 3, PH_DOWN = 4 };

struct Seg { int row, cnt, acc; };   // weight rows [row, row + cnt), accumulator slots from acc
struct GemvPlan {
  const char* w;      // matrix base
  int K, rt;          // row length, rows per tile
  int o0, n_local;    // outputs [o0, o0 + n_local) are this CTA's
  int nseg;
  Seg seg[6];
};

__device__ __forceinline__ void plan_gemv(const FusedDev& p, int ph, const char* lb, int cta, int grid, GemvPlan& g) {
  int n_out;
  if (ph == PH_QKV) { g.w = lb + p.off_wqkv; g.K = p.d; n_out = p.qkv_dim; }
  else if (ph == PH_O) { g.w = lb + p.off_wo; g.K = p.q_dim; n_out = p.d; }
  else if (ph == PH_GU) { g.w = lb + p.off_wgu; g.K = p.d; n_out = p.d_ffn; }
  else { g.w = lb + p.off_wd; g.K = p.d_ffn; n_out = p.d; }
  g.rt = min(F_RT, F_STAGE / (g.K * 2));
  g.o0 = (int)((int64_t)cta * n_out / grid);
  const int o1 = (int)((int64_t)(cta + 1) * n_out / grid);
  g.n_local = o1 - g.o0;
  if (ph != PH_GU) {
    g.nseg = 1;
    g.seg[0].row = g.o0; g.seg[0].cnt = g.n_local; g.seg[0].acc = 0;
    return;
  }
  // gate row of output o: (o / 128) * 256 + o % 128, its up row 128 further on
  g.nseg = 0;
  for (int b = g.o0 >> 7; b <= (o1 - 1) >> 7 && g.nseg < 6 && g.n_local > 0; ++b) {
    const int lo = max(g.o0, b << 7), hi = min(o1, (b + 1) << 7);
    g.seg[g.nseg].row = (b << 8) + (lo - (b << 7)); g.seg[g.nseg].cnt = hi - lo; g.seg[g.nseg].acc = lo - g.o0;
    ++g.nseg;
    g.seg[g.nseg].row = (b << 8) + 128 + (lo - (b << 7)); g.seg[g.nseg].cnt = hi - lo;
    g.seg[g.nseg].acc = g.n_local + lo - g.o0;
    ++g.nseg;
  }
}

struct AttPlan {
  int kvh, split;     // kvh < 0: this CTA has no part in the attention phase
  int j0, j1;         // cached positions [j0, j1) (never the new position)
  int n_tiles;
  bool owner;         // this CTA also takes the new position and appends it to the cache
};

__device__ __forceinline__ void plan_att(const FusedDev& p, int layer, int pos, int cta, AttPlan& a) {
  if (cta >= p.n_kv * p.splits) { a.kvh = -1; a.split = 0; a.j0 = a.j1 = 0; a.n_tiles = 0; a.owner = false; return; }
  a.kvh = cta % p.n_kv;
  a.split = cta / p.n_kv;
  const int l1 = layer + 1;
  const int win = (p.window > 0 && !(p.global_every > 0 && l1 % p.global_every == 0)) ? p.window : 0;
  const int lo = win > 0 ? max(0, pos + 1 - win) : 0;
  const int span = pos - lo;
  const int chunk = (span + p.splits - 1) / p.splits;
  a.j0 = min(pos, lo + a.split * chunk);
  a.j1 = min(pos, a.j0 + chunk);
  a.n_tiles = a.j1 > a.j0 ? (a.j1 - a.j0 + F_KEYS - 1) / F_KEYS : 0;
  a.owner = a.split == p.splits - 1;
}

struct Ring {
  uint32_t base;          // shared-memory address of stage 0
  uint64_t* full;         // [F_NS] a tile has landed
  uint64_t* empty;        // [F_NS] all consumer warps are done with it
  volatile int* s_abort;
};

// ------------------------------------------------------------------------------ producer warp
__device__ void fused_producer(const FusedDev& p, const Ring& rg, int pos) {
  const int lane = threadIdx.x & 31;
  const int cta = blockIdx.x, grid = gridDim.x;
  uint32_t tile_no = 0;
  bool dead = false, own_timeout = false;
  // lane 0 waits until the stage of tile `tile_no` is free again; every lane gets the answer
  auto acquire = [&]() -> bool {
    const uint32_t stage = tile_no % F_NS, use = tile_no / F_NS;
    int ok = 1;
    if (lane == 0) {
      if (*rg.s_abort) ok = 0;
      else if (use > 0 && !f_wait(&rg.empty[stage], (use - 1) & 1, rg.s_abort)) {
        ok = 0;
        if (!*rg.s_abort) own_timeout = true;
      }
    }
    return __shfl_sync(FULLMASK, ok, 0) != 0;
  };
  for (int li = 0; li < p.n_layers && !dead; ++li) {
    const int layer = p.layer_first + li;
    const char* lb = p.layer_base + (int64_t)layer * p.layer_stride;
    for (int ph = 0; ph < 5 && !dead; ++ph) {
      if (ph == PH_ATT) {
        AttPlan a;
        plan_att(p, layer, pos, cta, a);
        const bf16* kl = p.k_pool + (int64_t)layer * p.pool_layer_stride;
        const bf16* vl = p.v_pool + (int64_t)layer * p.pool_layer_stride;
        for (int t = 0; t < a.n_tiles; ++t) {
          if (!acquire()) { dead = true; break; }
          const uint32_t stage = tile_no % F_NS;
          const int jt = a.j0 + t * F_KEYS;
          const int nkeys = min(F_KEYS, a.j1 - jt);
          if (lane == 0) mbar_expect_tx(&rg.full[stage], (uint32_t)nkeys * 2u * (F_HD * 2));
          __syncwarp();
          for (int i = lane; i < nkeys; i += 32) {
            const int pk = jt + i;
            int page = p.block_table[pk / p.page_size];
            if ((unsigned)page >= (unsigned)p.num_pages) {
              atomicMin(p.status, (int)POP_E_INVALID);   // flagged; the copy below still completes, from page 0
              page = 0;
            }
            const int64_t off = (((int64_t)page * p.page_size + pk % p.page_size) * p.n_kv + a.kvh) * F_HD;
            const uint32_t dst = rg.base + stage * F_STAGE + i * F_PITCH;
            bulk_g2s(dst, kl + off, F_HD * 2, &rg.full[stage]);
            bulk_g2s(dst + F_KEYS * F_PITCH, vl + off, F_HD * 2, &rg.full[stage]);
          }
          ++tile_no;
        }
      } else {
        GemvPlan g;
        plan_gemv(p, ph, lb, cta, grid, g);
        for (int sg = 0; sg < g.nseg && !dead; ++sg) {
          for (int r0 = 0; r0 < g.seg[sg].cnt; r0 += g.rt) {
            if (!acquire()) { dead = true; break; }
            const uint32_t stage = tile_no % F_NS;
            const int nrows = min(g.rt, g.seg[sg].cnt - r0);
            const uint32_t bytes = (uint32_t)nrows * (uint32_t)g.K * 2u;
            if (lane == 0) {
              mbar_expect_tx(&rg.full[stage], bytes);
              bulk_g2s(rg.base + stage * F_STAGE, g.w + (int64_t)(g.seg[sg].row + r0) * g.K * 2, bytes, &rg.full[stage]);
            }
            ++tile_no;
          }
        }
      }
    }
  }
  if (dead && lane == 0) {
    if (own_timeout) f_fail(p, rg.s_abort);
    // copies still in flight must land before the CTA may exit: wait (bounded) for the fills of the
    // last F_NS tiles that were issued; a fill that completed earlier answers at once
    const uint32_t n = tile_no < (uint32_t)F_NS ? tile_no : (uint32_t)F_NS;
    for (uint32_t i = 0; i < n; ++i) {
      const uint32_t t = tile_no - 1 - i;
      const long long t0 = clock64();
      while (!mbar_try_wait(&rg.full[t % F_NS], (t / F_NS) & 1))
        if (clock64() - t0 > F_WAIT_CYCLES) break;
    }
  }
}

// ------------------------------------------------------------------------------ consumer: matrix-vector phase
struct ConsumerState {
  uint32_t tile_no;
  unsigned int bar_no;
  bool dead;
};

// waits (all lanes) for the fill of tile `tile_no`; false after a wait that ran out, for the whole warp
__device__ __forceinline__ bool tile_wait(const FusedDev& p, const Ring& rg, ConsumerState& cs) {
  if (cs.dead) return false;
  const uint32_t stage = cs.tile_no % F_NS, use = cs.tile_no / F_NS;
  const bool ok = __all_sync(FULLMASK, f_wait(&rg.full[stage], use & 1, rg.s_abort));
  if (!ok) {
    cs.dead = true;
    if ((threadIdx.x & 31) == 0) f_fail(p, rg.s_abort);
  }
  return ok;
}

// Grid-wide barrier of the consumer warps of all CTAs. False: the kernel is being abandoned.
__device__ bool grid_sync(const FusedDev& p, const Ring& rg, ConsumerState& cs) {
  if (consumer_bar_or(cs.dead)) return false;
  bool bad = false;
  if (threadIdx.x == 0) {
    const unsigned int target = (cs.bar_no + 1u) * gridDim.x;
    __threadfence();
    atomicAdd(p.sync, 1u);
    const long long t0 = clock64();
    unsigned int spins = 0;
    while (ld_acquire_gpu(p.sync) < target) {
      if ((++spins & 31u) == 0u) {
        if (ld_acquire_gpu(p.sync + 1) != 0u || *rg.s_abort) { bad = true; break; }
        if (clock64() - t0 > F_WAIT_CYCLES) { bad = true; f_fail(p, rg.s_abort); break; }
      }
      __nanosleep(20);
    }
    if (bad) *rg.s_abort = 1;
    __threadfence();
  }
  ++cs.bar_no;
  return !consumer_bar_or(bad);
}

template <bool NORM>
__device__ bool gemv_phase(const FusedDev& p, const Ring& rg, ConsumerState& cs, int ph, const char* lb, int cta,
                           float* acc, float* red) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  GemvPlan g;
  plan_gemv(p, ph, lb, cta, gridDim.x, g);
  const int steps = g.K >> 8;
  const int nj = steps > warp ? (steps - warp + FW - 1) / FW : 0;
  // this lane's part of the activation vector: elements ((j FW + warp) 256 + 8 lane) .. + 7
  float xs[F_MAXJ][8];
  if (NORM) {
    const float* gain = reinterpret_cast<const float*>(lb + (ph == PH_QKV ? p.off_ln_in : p.off_ln_ffn));
    float ss = 0.f;
    for (int c = tid * 4; c < p.d; c += FW * 32 * 4) {
      const float4 v = __ldcg(reinterpret_cast<const float4*>(p.xb + c));
      ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    ss = f_warp_sum(ss);
    if (lane == 0) red[warp] = ss;
    if (consumer_bar_or(cs.dead)) return false;
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < FW; ++w) tot += red[w];
    const float rstd = rsqrtf(tot / (float)p.d + p.eps);
#pragma unroll
    for (int j = 0; j < F_MAXJ; ++j) {
      if (j < nj) {
        const int k = ((j * FW + warp) << 8) + lane * 8;
        const float4 a0 = __ldcg(reinterpret_cast<const float4*>(p.xb + k));
        const float4 a1 = __ldcg(reinterpret_cast<const float4*>(p.xb + k + 4));
        const float4 g0 = *reinterpret_cast<const float4*>(gain + k);
        const float4 g1 = *reinterpret_cast<const float4*>(gain + k + 4);
        xs[j][0] = bf16_round(a0.x * rstd * g0.x); xs[j][1] = bf16_round(a0.y * rstd * g0.y);
        xs[j][2] = bf16_round(a0.z * rstd * g0.z); xs[j][3] = bf16_round(a0.w * rstd * g0.w);
        xs[j][4] = bf16_round(a1.x * rstd * g1.x); xs[j][5] = bf16_round(a1.y * rstd * g1.y);
        xs[j][6] = bf16_round(a1.z * rstd * g1.z); xs[j][7] = bf16_round(a1.w * rstd * g1.w);
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) xs[j][e] = 0.f;
      }
    }
  } else {
    const bf16* xsrc = ph == PH_O ? p.ob : p.ab;
#pragma unroll
    for (int j = 0; j < F_MAXJ; ++j) {
      if (j < nj) {
        const int k = ((j * FW + warp) << 8) + lane * 8;
        const uint4 raw = __ldcg(reinterpret_cast<const uint4*>(xsrc + k));
        f_unpack8(raw, xs[j]);
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) xs[j][e] = 0.f;
      }
    }
  }
  const uint32_t rowb = (uint32_t)g.K * 2u;
  for (int sg = 0; sg < g.nseg; ++sg) {
    for (int r0 = 0; r0 < g.seg[sg].cnt; r0 += g.rt) {
      const int nrows = min(g.rt, g.seg[sg].cnt - r0);
      if (tile_wait(p, rg, cs)) {
        const uint32_t stage = cs.tile_no % F_NS;
        const uint32_t sb = rg.base + stage * F_STAGE + warp * 512 + lane * 16;
        for (int r = 0; r < nrows; r += 4) {
          const int nq = min(4, nrows - r);
          float a[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int j = 0; j < F_MAXJ; ++j) {
            if (j < nj) {
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                if (q < nq) {
                  float wf[8];
                  f_unpack8(lds128(sb + (uint32_t)(r + q) * rowb + (uint32_t)j * (FW * 512)), wf);
#pragma unroll
                  for (int e = 0; e < 8; ++e) a[q] = fmaf(wf[e], xs[j][e], a[q]);
                }
              }
            }
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (q < nq) {
              const float v = f_warp_sum(a[q]);
              if (lane == 0) acc[(g.seg[sg].acc + r0 + r + q) * FW + warp] = v;
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&rg.empty[stage]);
      }
      ++cs.tile_no;
    }
  }
  if (consumer_bar_or(cs.dead)) return false;
  for (int t = tid; t < g.n_local; t += FW * 32) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < FW; ++w) v += acc[t * FW + w];
    const int o = g.o0 + t;
    if (ph == PH_QKV) {
      p.qkv[o] = v;
    } else if (ph == PH_GU) {
      float u = 0.f;
#pragma unroll
      for (int w = 0; w < FW; ++w) u += acc[(g.n_local + t) * FW + w];
      p.ab[o] = __float2bfloat16_rn(f_act(v, p.act) * u);
    } else {
      p.xb[o] = __ldcg(p.xb + o) + v;
    }
  }
  return true;
}

// ------------------------------------------------------------------------------ consumer: attention phase
// Scratch during the tile loop: the one-key tile of the new position (16 K rows, then 16 V rows, at
// F_PITCH) and the group's roped queries; after it: the merge of the four key groups, then the split
// weights of the last CTA's merge.
constexpr int F_XT_BYTES = 2 * 16 * F_PITCH;
static_assert(F_XT_BYTES + F_MAXG * F_HD * 2 <= F_SCRATCH, "new-position tile and queries fit the scratch");
static_assert((2 * 4 * F_MAXG + 4 * F_MAXG * F_HD) * 4 <= F_SCRATCH, "group merge fits the scratch");
static_assert((F_MAXG * 64 + F_MAXG) * 4 <= F_SCRATCH, "split weights fit the scratch");

__device__ bool att_phase(const FusedDev& p, const Ring& rg, ConsumerState& cs, int layer, int pos, const char* lb,
                          int cta, uint8_t* scratch, int* s_flag) {
  AttPlan a;
  plan_att(p, layer, pos, cta, a);
  if (a.kvh < 0) return true;
  constexpr int NT = F_HD / 16;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.n_q / p.n_kv;
  uint8_t* xt = scratch;
  bf16* q_s = reinterpret_cast<bf16*>(scratch + F_XT_BYTES);
  const uint32_t xt_u32 = smem_u32(xt);

  // ---- the new position: per-head norm, RoPE; queries to shared memory, key and value to the
  // one-key tile and (owner CTA of the kv head) to the cache
  int page_new = p.block_table[pos / p.page_size];
  const bool page_ok = (unsigned)page_new < (unsigned)p.num_pages;
  if (!page_ok && a.owner && tid == 0) atomicMin(p.status, (int)POP_E_INVALID);   // nothing is written for it
  if (a.owner) {
    // rows 1..15 of both halves of the one-key tile are zeros
    for (int i = tid; i < 2 * 15 * 16; i += FW * 32) {
      const int half = i / (15 * 16), rem = i - half * 15 * 16;
      const int row = 1 + rem / 16, c = rem % 16;
      *reinterpret_cast<uint4*>(xt + half * 16 * F_PITCH + row * F_PITCH + c * 16) = make_uint4(0, 0, 0, 0);
    }
  }
  for (int it = warp; it < G + 2; it += FW) {
    const bool is_q = it < G, is_k = it == G;
    if (!is_q && !a.owner) continue;
    const float* src = p.qkv + (is_q ? (int64_t)(a.kvh * G + it) * F_HD
                                     : (is_k ? (int64_t)p.q_dim + a.kvh * F_HD
                                             : (int64_t)p.q_dim + p.kv_dim + a.kvh * F_HD));
    float lo[2], hi[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      lo[u] = __ldcg(src + lane + 32 * u);
      hi[u] = __ldcg(src + lane + 32 * u + F_HD / 2);
    }
    if (is_q || is_k) {
      if (p.qk_norm) {
        const float* gain = reinterpret_cast<const float*>(lb + (is_q ? p.off_qn : p.off_kn));
        float ss = 0.f;
#pragma unroll
        for (int u = 0; u < 2; ++u) ss += lo[u] * lo[u] + hi[u] * hi[u];
        ss = f_warp_sum(ss);
        const float rstd = rsqrtf(ss / (float)F_HD + p.eps);
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          lo[u] = lo[u] * rstd * gain[lane + 32 * u];
          hi[u] = hi[u] * rstd * gain[lane + 32 * u + F_HD / 2];
        }
      }
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const float2 csn = p.rope_row[lane + 32 * u];
        const float x = lo[u] * csn.x - hi[u] * csn.y;
        const float y = hi[u] * csn.x + lo[u] * csn.y;
        lo[u] = x;
        hi[u] = y;
      }
    }
    bf16* dst_s = is_q ? q_s + it * F_HD : reinterpret_cast<bf16*>(xt + (is_k ? 0 : 16 * F_PITCH));
    bf16* dst_g = nullptr;
    if (!is_q && page_ok) {
      bf16* pool = (is_k ? p.k_pool : p.v_pool) + (int64_t)layer * p.pool_layer_stride;
      dst_g = pool + (((int64_t)page_new * p.page_size + pos % p.page_size) * p.n_kv + a.kvh) * F_HD;
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const bf16 l = __float2bfloat16_rn(lo[u]), h = __float2bfloat16_rn(hi[u]);
      dst_s[lane + 32 * u] = l;
      dst_s[lane + 32 * u + F_HD / 2] = h;
      if (dst_g) {
        dst_g[lane + 32 * u] = l;
        dst_g[lane + 32 * u + F_HD / 2] = h;
      }
    }
  }
  if (consumer_bar_or(cs.dead)) return false;

  // Q^T as the B operand: thread holds head lane/4, dims 16 ks + 2 (lane%4) + {0, 1} and + 8
  uint32_t qb[NT][2];
  {
    const int g = lane >> 2;
    const bf16* qrow = q_s + (g < G ? g : 0) * F_HD + (lane & 3) * 2;
#pragma unroll
    for (int ks = 0; ks < NT; ++ks) {
      qb[ks][0] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16) : 0u;
      qb[ks][1] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8) : 0u;
    }
  }
  // warp = 2 * group + half: the two warps of a group of 16 keys both form its scores; each
  // accumulates one half of the head dimension
  const int grp = warp >> 1, half = warp & 1;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  float o[NT / 2][4];
#pragma unroll
  for (int t = 0; t < NT / 2; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;
  const int mi = lane >> 3, r8 = lane & 7, kr = lane >> 2;

  // one group of 16 keys (gvalid >= 1 of them real) at shared addresses stK / stV
  auto do_group = [&](uint32_t stK, uint32_t stV, int gvalid) {
    float s[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
    const uint32_t k_lane = stK + ((mi & 1) * 8 + r8) * F_PITCH + (mi >> 1) * 16;
#pragma unroll
    for (int ks = 0; ks < NT; ks += 2) {
      uint32_t a0[4], a1[4];
      f_ldsm_x4(a0, k_lane + (2 * ks) * 16);
      f_ldsm_x4(a1, k_lane + (2 * ks + 2) * 16);
      f_mma_16816(s, a0, qb[ks][0], qb[ks][1]);
      f_mma_16816(sb, a1, qb[ks + 1][0], qb[ks + 1][1]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) s[i] += sb[i];
    const bool v0 = kr < gvalid, v1 = kr + 8 < gvalid;
    const float s0 = v0 ? s[0] * p.scale_log2 : -INFINITY, s1 = v0 ? s[1] * p.scale_log2 : -INFINITY;
    const float s2 = v1 ? s[2] * p.scale_log2 : -INFINITY, s3 = v1 ? s[3] * p.scale_log2 : -INFINITY;
    float x0 = fmaxf(s0, s2), x1 = fmaxf(s1, s3);
#pragma unroll
    for (int w = 4; w < 32; w <<= 1) {
      x0 = fmaxf(x0, __shfl_xor_sync(FULLMASK, x0, w));
      x1 = fmaxf(x1, __shfl_xor_sync(FULLMASK, x1, w));
    }
    const float n0 = fmaxf(m0, x0), n1 = fmaxf(m1, x1);       // finite: key 0 of the group is real
    const float f0 = exp2f(m0 - n0), f1 = exp2f(m1 - n1);
    const float p0 = exp2f(s0 - n0), p1 = exp2f(s1 - n1), p2 = exp2f(s2 - n0), p3 = exp2f(s3 - n1);
    l0 = l0 * f0 + (p0 + p2);
    l1 = l1 * f1 + (p1 + p3);
    m0 = n0;
    m1 = n1;
    if (__any_sync(FULLMASK, f0 != 1.f || f1 != 1.f)) {
#pragma unroll
      for (int t = 0; t < NT / 2; ++t) {
        o[t][0] *= f0; o[t][1] *= f1; o[t][2] *= f0; o[t][3] *= f1;
      }
    }
    const uint32_t pb0 = f_movm_t(f_pack_bf16x2(p0, p1));
    const uint32_t pb1 = f_movm_t(f_pack_bf16x2(p2, p3));
    const uint32_t v_lane = stV + ((mi >> 1) * 8 + r8) * F_PITCH + (mi & 1) * 16;
#pragma unroll
    for (int t = 0; t < NT / 2; ++t) {
      uint32_t av[4];
      f_ldsm_x4_t(av, v_lane + (2 * (half * (NT / 2) + t)) * 16);
      f_mma_16816(o[t], av, pb0, pb1);
    }
  };

  for (int t = 0; t < a.n_tiles; ++t) {
    const int nkeys = min(F_KEYS, a.j1 - (a.j0 + t * F_KEYS));
    if (tile_wait(p, rg, cs)) {
      const uint32_t stage = cs.tile_no % F_NS;
      const uint32_t stK = rg.base + stage * F_STAGE + grp * 16 * F_PITCH;
      const uint32_t stV = stK + F_KEYS * F_PITCH;
      const int gvalid = min(16, nkeys - grp * 16);
      if (gvalid > 0) {
        if (gvalid < 16) {
          // value rows past the range hold whatever the stage held before: this warp clears the part
          // it is going to multiply by zero weights
          for (int i = lane; i < 16 * 8; i += 32) {
            const int row = i >> 3, c = i & 7;
            if (row >= gvalid)
              asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(stV + row * F_PITCH + half * 128 + c * 16),
                           "r"(0u)
                           : "memory");
          }
          __syncwarp();
        }
        do_group(stK, stV, gvalid);
        if (gvalid < 16) fence_proxy_async_smem();   // the stage's next fill must come after these stores
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&rg.empty[stage]);
    }
    ++cs.tile_no;
  }
  if (a.owner && grp == 0 && !cs.dead) do_group(xt_u32, xt_u32 + 16 * F_PITCH, 1);

#pragma unroll
  for (int w = 4; w < 32; w <<= 1) {
    l0 += __shfl_xor_sync(FULLMASK, l0, w);
    l1 += __shfl_xor_sync(FULLMASK, l1, w);
  }
  if (consumer_bar_or(cs.dead)) return false;      // queries and the one-key tile are no longer needed
  float* sm_m = reinterpret_cast<float*>(scratch);   // [4][8]
  float* sm_l = sm_m + 4 * F_MAXG;                   // [4][8]
  float* sm_o = sm_l + 4 * F_MAXG;                   // [4][8][F_HD]
  {
    const int h0 = (lane & 3) * 2;
    if (half == 0 && lane < 4) {
      sm_m[grp * F_MAXG + h0] = m0; sm_m[grp * F_MAXG + h0 + 1] = m1;
      sm_l[grp * F_MAXG + h0] = l0; sm_l[grp * F_MAXG + h0 + 1] = l1;
    }
    float* so = sm_o + (grp * F_MAXG + h0) * F_HD + half * (F_HD / 2);
#pragma unroll
    for (int t = 0; t < NT / 2; ++t) {
      so[t * 16 + kr] = o[t][0];
      so[F_HD + t * 16 + kr] = o[t][1];
      so[t * 16 + kr + 8] = o[t][2];
      so[F_HD + t * 16 + kr + 8] = o[t][3];
    }
  }
  consumer_bar_or(false);
  for (int idx = tid; idx < G * F_HD; idx += FW * 32) {
    const int g = idx / F_HD, e = idx - g * F_HD;
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < 4; ++w) mm = fmaxf(mm, sm_m[w * F_MAXG + g]);
    float ll = 0.f, oo = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float mw = sm_m[w * F_MAXG + g];
      const float f = (mw == -INFINITY) ? 0.f : exp2f(mw - mm);
      ll += sm_l[w * F_MAXG + g] * f;
      oo += sm_o[(w * F_MAXG + g) * F_HD + e] * f;
    }
    float* dst = p.partial + ((int64_t)(a.kvh * G + g) * p.splits + a.split) * (F_HD + 2);
    dst[2 + e] = oo;
    if (e == 0) {
      dst[0] = mm;
      dst[1] = ll;
    }
  }
  // the last CTA of this kv head to get here merges the splits; the counter wraps back to zero
  __threadfence();
  consumer_bar_or(false);
  if (tid == 0) {
    const unsigned int old = atomicInc(p.counters + a.kvh, (unsigned int)p.splits - 1u);
    *s_flag = old == (unsigned int)p.splits - 1u;
  }
  consumer_bar_or(false);
  if (!*reinterpret_cast<volatile int*>(s_flag)) return true;
  __threadfence();
  float* wgt = reinterpret_cast<float*>(scratch);     // [G][64]
  float* inv_l = wgt + F_MAXG * 64;                   // [G]
  for (int g = warp; g < G; g += FW) {
    const float* src = p.partial + (int64_t)(a.kvh * G + g) * p.splits * (F_HD + 2);
    const int s0 = lane, s1 = lane + 32;
    const float ma = s0 < p.splits ? __ldcg(src + s0 * (F_HD + 2)) : -INFINITY;
    const float mb = s1 < p.splits ? __ldcg(src + s1 * (F_HD + 2)) : -INFINITY;
    const float la = s0 < p.splits ? __ldcg(src + s0 * (F_HD + 2) + 1) : 0.f;
    const float lbb = s1 < p.splits ? __ldcg(src + s1 * (F_HD + 2) + 1) : 0.f;
    float mm = fmaxf(ma, mb);
#pragma unroll
    for (int w = 16; w > 0; w >>= 1) mm = fmaxf(mm, __shfl_xor_sync(FULLMASK, mm, w));
    const float wa = (ma == -INFINITY) ? 0.f : exp2f(ma - mm);
    const float wb = (mb == -INFINITY) ? 0.f : exp2f(mb - mm);
    wgt[g * 64 + s0] = wa;
    wgt[g * 64 + s1] = wb;
    const float ll = f_warp_sum(la * wa + lbb * wb);
    if (lane == 0) inv_l[g] = 1.0f / ll;
  }
  consumer_bar_or(false);
  for (int idx = tid; idx < G * F_HD; idx += FW * 32) {
    const int g = idx / F_HD, e = idx - g * F_HD;
    const float* src = p.partial + (int64_t)(a.kvh * G + g) * p.splits * (F_HD + 2) + 2 + e;
    float oo = 0.f;
#pragma unroll 6
    for (int sp = 0; sp < p.splits; ++sp) oo = fmaf(__ldcg(src + sp * (F_HD + 2)), wgt[g * 64 + sp], oo);
    p.ob[(int64_t)(a.kvh * G + g) * F_HD + e] = __float2bfloat16_rn(oo * inv_l[g]);
  }
  return true;
}

// ------------------------------------------------------------------------------ kernel
__global__ void __launch_bounds__(F_THREADS, 1) decode_fused_kernel(const FusedDev p) {
  extern __shared__ __align__(128) uint8_t fsm[];
  uint8_t* scratch = fsm + F_NS * F_STAGE;
  uint64_t* full = reinterpret_cast<uint64_t*>(scratch + F_SCRATCH);
  uint64_t* empty = full + F_NS;
  float* red = reinterpret_cast<float*>(empty + F_NS);      // [FW]
  int* s_abort = reinterpret_cast<int*>(red + FW);
  int* s_flag = s_abort + 1;
  uint32_t* s_raised = reinterpret_cast<uint32_t*>(s_abort + 2);
  if (status_raised(p.status, s_raised)) return;
  if (threadIdx.x == 0) {
    for (int i = 0; i < F_NS; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], FW);
    }
    *s_abort = 0;
    fence_barrier_init();
  }
  __syncthreads();
  const int pos = p.pos_dev ? *p.pos_dev : p.pos;
  Ring rg;
  rg.base = smem_u32(fsm);
  rg.full = full;
  rg.empty = empty;
  rg.s_abort = s_abort;
  const int cta = blockIdx.x;
  if ((threadIdx.x >> 5) == FW) {
    fused_producer(p, rg, pos);
  } else {
    ConsumerState cs;
    cs.tile_no = 0;
    cs.bar_no = 0;
    cs.dead = false;
    float* acc = reinterpret_cast<float*>(scratch);
    bool ok = true;
    for (int li = 0; li < p.n_layers && ok; ++li) {
      const int layer = p.layer_first + li;
      const char* lb = p.layer_base + (int64_t)layer * p.layer_stride;
      ok = gemv_phase<true>(p, rg, cs, PH_QKV, lb, cta, acc, red) && grid_sync(p, rg, cs);
      ok = ok && att_phase(p, rg, cs, layer, pos, lb, cta, scratch, s_flag) && grid_sync(p, rg, cs);
      ok = ok && gemv_phase<false>(p, rg, cs, PH_O, lb, cta, acc, red) && grid_sync(p, rg, cs);
      ok = ok && gemv_phase<true>(p, rg, cs, PH_GU, lb, cta, acc, red) && grid_sync(p, rg, cs);
      ok = ok && gemv_phase<false>(p, rg, cs, PH_DOWN, lb, cta, acc, red);
      if (ok && li + 1 < p.n_layers) ok = grid_sync(p, rg, cs);
    }
    if (!ok && (threadIdx.x & 31) == 0) *s_abort = 1;    // the producer stops at its next tile
  }
  __syncthreads();
}

int g_fused_sms = 0;         // 0: not looked at yet; < 0: the kernel cannot be used on this device

int fused_grid() {
  if (g_fused_sms != 0) return g_fused_sms;
  int dev = 0, n = 0, coop = 0, per_sm = 0;
  g_fused_sms = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return -1;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return -1;
  if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return -1;
  if (cudaFuncSetAttribute(decode_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, F_SMEM) != cudaSuccess ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_fused_kernel, F_THREADS, F_SMEM) != cudaSuccess ||
      per_sm < 1) {
    cudaGetLastError();
    return -1;
  }
  g_fused_sms = n;
  return n;
}

}  // namespace

// Shapes the kernel covers: one sequence, head_dim 128, bf16 weights, no post-norms, every K (d_model,
// q_dim, d_ffn) a multiple of 256 and at most 16384, and a group of at most 8 query heads per kv head.
// POP_DECODE_FUSED=0 in the environment keeps the chain of single kernels.
bool decode_fused_supported(const pop_config_t& c, int batch, bool fp8) {
  static const bool enabled = [] {
    const char* e = getenv("POP_DECODE_FUSED");
    return !(e && e[0] == '0');
  }();
  const char* now = getenv("POP_DECODE_FUSED");      // a later "0" still wins (A/B runs in one process)
  if (!enabled || (now && now[0] == '0')) return false;
  if (batch != 1 || fp8 || c.post_norms || c.head_dim != F_HD) return false;
  if (c.n_kv_heads < 1 || c.n_q_heads % c.n_kv_heads || c.n_q_heads / c.n_kv_heads > F_MAXG) return false;
  const int q_dim = c.n_q_heads * c.head_dim;
  const int ks[3] = {c.d_model, q_dim, c.d_ffn};
  for (int k : ks)
    if (k % 256 || k > F_MAXJ * FW * 256 || k * 2 > F_STAGE) return false;
  const int grid = fused_grid();
  if (grid < 1 || c.n_kv_heads > grid) return false;
  const int qkv_dim = q_dim + 2 * c.n_kv_heads * c.head_dim;
  // accumulator slots of one CTA: its outputs (twice for the gated phase)
  const int most = 2 * (c.d_ffn / grid + 2);
  if (most > F_MAXACC || qkv_dim / grid + 2 > F_MAXACC || c.d_ffn / grid + 2 > 256) return false;
  return true;
}

int launch_decode_fused(const FusedDecodeArgs& a, cudaStream_t s) {
  const int grid = fused_grid();
  if (grid < 1) return POP_E_CUDA;
  if (!a.layer_base || !a.xb || !a.qkv || !a.ob || !a.ab || !a.partial || !a.rope_row || !a.k_pool || !a.v_pool ||
      !a.block_table || !a.counters || !a.sync || a.n_layers < 1 || a.num_pages < 1 || a.page_size < 1)
    return POP_E_INVALID;
  FusedDev p = a;
  p.status = status_word();
  if (!p.status) return POP_E_CUDA;
  p.splits = grid / a.n_kv;
  if (p.splits > 64) p.splits = 64;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)F_HD);
  void* args[1] = {&p};
  if (cudaLaunchCooperativeKernel((const void*)decode_fused_kernel, dim3(grid), dim3(F_THREADS), args, (size_t)F_SMEM, s) !=
      cudaSuccess) {
    cudaGetLastError();
    return POP_E_CUDA;
  }
  count_launch();
  return POP_OK;
}

}  // namespace pop
