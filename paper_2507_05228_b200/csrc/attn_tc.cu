// Attention-pass on the 5th-generation tensor cores (tcgen05 + TMEM) for bf16, head_dim 128.
//
// One CTA = one tile of up to 128 query slots of one query shard, one head, and either one KV shard
// (partials: Algorithm 3 for the pair) or all KV shards one after another (fused: the post-pass carry
// n, w, o of Algorithm 4 is the running max / sum / output of the streaming softmax).
//
// Warp roles (9 warps):
//   0-3  softmax: thread r owns query row r = TMEM lane r; reads the logits tile S with tcgen05.ld, applies the
//        shard mask (row r sees the first vis[r][k] keys of the shard), keeps running max / sum, writes the
//        probabilities P (bf16) into shared memory in the 128-byte-swizzled K-major layout, rescales the output
//        accumulator in TMEM when the running max moved by more than 2^8, and runs the epilogue.
//   4    MMA issuer (one lane): S = Q K^T  (M128 N128 K16 x 8) and O += P V (M128 N128 K16 x 8), accumulators
//        in TMEM (S double-buffered at columns 0/128, O at column 256); completion via tcgen05.commit.
//   5-6  K loader, 7-8 V loader: index-mapped gather of 256-byte rows with 16-byte cp.async into the swizzled
//        layout the MMA descriptors expect; rows past the visible prefix are zero-filled.
// Every mbarrier wait is bounded: on expiry the CTA raises a flag, records a code in the plan's status word
// and drains without waiting again.
#include "cascade_internal.cuh"

namespace cascade {
namespace tc {

constexpr int kThreads = 288;
constexpr int kTile = 128;                 // query rows per CTA and keys per KV tile
constexpr int kD = 128;                    // head_dim
constexpr int kTileBytes = kTile * kD * 2; // 32 KiB, laid out [2 halves][128 rows][128 bytes]
constexpr int kHalfBytes = kTileBytes / 2;
constexpr int kStages = 2;
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.f;   // log2 units

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + kTileBytes;
constexpr int kOffV = kOffK + kStages * kTileBytes;
constexpr int kOffP = kOffV + kStages * kTileBytes;
constexpr int kOffBar = kOffP + kTileBytes;
constexpr int kNumBars = 16;
constexpr int kOffMisc = kOffBar + kNumBars * 8;
constexpr int kSmemBytes = kOffMisc + 64 + 1024;  // + alignment slack

enum Bar { Q_FULL = 0, K_FULL = 1, K_EMPTY = 3, V_FULL = 5, V_EMPTY = 7, S_FULL = 9, S_EMPTY = 11, P_FULL = 13,
           P_EMPTY = 14 };

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

struct WaitCtx {
  volatile int* abort_flag;  // shared memory
  int32_t* status;           // global
};

// Bounded wait: gives up after ~2 s, raises the CTA's abort flag and records `code`.
__device__ __noinline__ bool wait_slow(const WaitCtx& c, uint32_t bar, uint32_t parity, int code) {
  const uint64_t t0 = global_timer_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*c.abort_flag || *reinterpret_cast<volatile int32_t*>(c.status) != 0) return false;
      if (global_timer_ns() - t0 > 2000000000ull) {
        *c.abort_flag = 1;
        atomicCAS(c.status, 0, code);
        return false;
      }
    }
  }
  return true;
}
__device__ __forceinline__ bool wait_bar(const WaitCtx& c, uint32_t bar, uint32_t parity, int code) {
  if (*c.abort_flag) return false;
  if (mbar_try_wait(bar, parity)) return true;
  return wait_slow(c, bar, parity, code);
}

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle.  Fields: start address >> 4 (bits 0-13), leading-dimension
// byte offset >> 4 (16-29), stride-dimension byte offset >> 4 (32-45), descriptor version 1 (46-47), layout
// type 2 = SWIZZLE_128B (61-63).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
         ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor for kind::f16: D fp32 (bits 4-5 = 1), A and B bf16 (bits 7-9, 10-12 = 1), operand
// majors (bit 15 A, bit 16 B; 0 = K-major, 1 = MN-major), N >> 3 at bits 17-22, M >> 4 at bits 24-28.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n, int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

#define CASCADE_TMEM_LD32(taddr, r, o)                                                                         \
  asm volatile(                                                                                                 \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                                 \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "                                 \
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"                \
      : "=r"(r[o + 0]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]),         \
        "=r"(r[o + 6]), "=r"(r[o + 7]), "=r"(r[o + 8]), "=r"(r[o + 9]), "=r"(r[o + 10]), "=r"(r[o + 11]),       \
        "=r"(r[o + 12]), "=r"(r[o + 13]), "=r"(r[o + 14]), "=r"(r[o + 15]), "=r"(r[o + 16]), "=r"(r[o + 17]),   \
        "=r"(r[o + 18]), "=r"(r[o + 19]), "=r"(r[o + 20]), "=r"(r[o + 21]), "=r"(r[o + 22]), "=r"(r[o + 23]),   \
        "=r"(r[o + 24]), "=r"(r[o + 25]), "=r"(r[o + 26]), "=r"(r[o + 27]), "=r"(r[o + 28]), "=r"(r[o + 29]),   \
        "=r"(r[o + 30]), "=r"(r[o + 31])                                                                        \
      : "r"(taddr)                                                                                              \
      : "memory")

#define CASCADE_TMEM_ST32(taddr, r, o)                                                                         \
  asm volatile(                                                                                                 \
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "                                                          \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "                                 \
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"                       \
      ::"r"(r[o + 0]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]),               \
        "r"(r[o + 6]), "r"(r[o + 7]), "r"(r[o + 8]), "r"(r[o + 9]), "r"(r[o + 10]), "r"(r[o + 11]),             \
        "r"(r[o + 12]), "r"(r[o + 13]), "r"(r[o + 14]), "r"(r[o + 15]), "r"(r[o + 16]), "r"(r[o + 17]),         \
        "r"(r[o + 18]), "r"(r[o + 19]), "r"(r[o + 20]), "r"(r[o + 21]), "r"(r[o + 22]), "r"(r[o + 23]),         \
        "r"(r[o + 24]), "r"(r[o + 25]), "r"(r[o + 26]), "r"(r[o + 27]), "r"(r[o + 28]), "r"(r[o + 29]),         \
        "r"(r[o + 30]), "r"(r[o + 31]), "r"(taddr)                                                              \
      : "memory")

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {  // 2^x, MUFU; ex2(-inf) = +0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Byte offset of 16-byte chunk `chunk` (0..15) of row `row` inside a [2][128][128 B] swizzled tile.
__device__ __forceinline__ uint32_t tile_offset(int row, int chunk) {
  return (uint32_t)((chunk >> 3) * kHalfBytes + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

// Gather up to 128 rows (row i of the tile = token idx[i], i < n_valid; the rest zero-filled) with `nthr` threads.
__device__ __forceinline__ void gather_tile(uint32_t tile_saddr, const __nv_bfloat16* base, int64_t token_stride,
                                            const int32_t* idx, int n_valid, int t, int nthr) {
  const int chunk = t & 15;
  const int rows_per_pass = nthr >> 4;
  for (int row = t >> 4; row < kTile; row += rows_per_pass) {
    const bool ok = row < n_valid;
    const int64_t tok = ok ? __ldg(idx + row) : 0;
    cp_async16(tile_saddr + tile_offset(row, chunk), base + tok * token_stride + chunk * 8, ok ? 16u : 0u);
  }
}

__global__ void __launch_bounds__(kThreads, 1) attn_tc_kernel(AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar0 = smem_base + kOffBar;
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffMisc + 4);

  const PlanDev& pl = p.plan;
  const int P = pl.n_kv_shards;
  const int n_parts = p.fused ? 1 : P;
  const int b = blockIdx.z / n_parts;
  const int part = blockIdx.z % n_parts;
  const int map = pl.n_maps == 1 ? 0 : b;
  const int h = blockIdx.y;
  const int g = h / p.G;
  const int4 qt = pl.qtiles128[(size_t)map * pl.n_qtiles128 + blockIdx.x];
  const int row0 = qt.x, nrows = qt.y;
  if (nrows == 0) return;  // padding entry (uniform for the CTA)
  if (*reinterpret_cast<volatile int32_t*>(pl.status) != 0) return;  // an earlier CTA gave up: do not pile on
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int32_t* q_idx = pl.q_idx + (size_t)map * pl.n_q;
  const int32_t* kv_idx = pl.kv_idx + (size_t)map * pl.n_kv;
  const int32_t* kv_off = pl.kv_off + (size_t)map * (P + 1);
  const int32_t* vis = pl.vis + (size_t)map * pl.n_q * P;
  const int32_t* vis_last = vis + (size_t)(row0 + nrows - 1) * P;  // longest prefix of the tile (rows ascend)
  const int32_t* vis_first = vis + (size_t)row0 * P;               // shortest prefix
  const int k_begin = p.fused ? 0 : part, k_end = p.fused ? P : part + 1;
  WaitCtx wc{abort_flag, pl.status};

  if (tid == 0) {
    mbar_init(bar(Q_FULL), 64);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar(K_FULL + s), 64);
      mbar_init(bar(K_EMPTY + s), 1);
      mbar_init(bar(V_FULL + s), 64);
      mbar_init(bar(V_EMPTY + s), 1);
      mbar_init(bar(S_FULL + s), 1);
      mbar_init(bar(S_EMPTY + s), 128);
    }
    mbar_init(bar(P_FULL), 128);
    mbar_init(bar(P_EMPTY), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_base + (uint32_t)kOffMisc),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp < 4) {
    // ------------------------------------------------------------------ softmax + epilogue
    const int r = tid;  // query row of the tile = TMEM lane
    const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
    const float c = p.scale * 1.4426950408889634f;  // logits are kept in log2 units: x = s * scale * log2(e)
    float m_run = -INFINITY;   // reference max the accumulators are scaled by (may lag by < 2^8)
    float m_true = -INFINITY;  // exact running max
    float l_run = 0.f;
    int i = 0;  // flattened KV tile counter
    const bool row_ok = r < nrows;
    for (int kk = k_begin; kk < k_end; ++kk) {
      const int need = __ldg(vis_last + kk);
      const int full_upto = __ldg(vis_first + kk);
      const int my_vis = row_ok ? __ldg(vis + (size_t)(row0 + r) * P + kk) : 0;
      for (int t0 = 0; t0 < need; t0 += kTile, ++i) {
        const int sb = i & 1;
        wait_bar(wc, bar(S_FULL + sb), (uint32_t)((i >> 1) & 1), 1);
        tc_fence_after();
        uint32_t sr[128];
        const uint32_t s_addr = lane_base + (uint32_t)(sb * 128);
        CASCADE_TMEM_LD32(s_addr, sr, 0);
        CASCADE_TMEM_LD32(s_addr + 32, sr, 32);
        CASCADE_TMEM_LD32(s_addr + 64, sr, 64);
        CASCADE_TMEM_LD32(s_addr + 96, sr, 96);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(bar(S_EMPTY + sb));  // logits are in registers: the buffer may be overwritten
        // mask (only tiles that reach past the shortest prefix of the CTA need it) and tile max
        float tmax = -INFINITY;
        if (t0 + kTile <= full_upto) {
#pragma unroll
          for (int j = 0; j < 128; ++j) tmax = fmaxf(tmax, __uint_as_float(sr[j]));
        } else {
          const int lim = my_vis - t0;  // columns [0, lim) are visible to this row
#pragma unroll
          for (int j = 0; j < 128; ++j) {
            if (j >= lim) sr[j] = 0xff800000u;  // -inf
            tmax = fmaxf(tmax, __uint_as_float(sr[j]));
          }
        }
        tmax *= c;
        m_true = fmaxf(m_true, tmax);
        float m_new = m_run;
        if (m_run == -INFINITY || m_true > m_run + kRescaleThreshold) m_new = m_true;
        const float alpha = (m_run == -INFINITY) ? 0.f : ex2(m_run - m_new);
        const bool changed = m_new != m_run;
        m_run = m_new;
        const float neg_m = (m_run == -INFINITY) ? 0.f : -m_run;
        float psum = 0.f;
        uint32_t pk[64];
#pragma unroll
        for (int j = 0; j < 128; j += 2) {
          const float p0 = ex2(fmaf(__uint_as_float(sr[j]), c, neg_m));
          const float p1 = ex2(fmaf(__uint_as_float(sr[j + 1]), c, neg_m));
          psum += p0 + p1;
          pk[j >> 1] = pack_bf16x2(p0, p1);
        }
        l_run = l_run * alpha + psum;
        // P buffer free and O quiescent once the previous PV product has completed
        if (i > 0) {
          wait_bar(wc, bar(P_EMPTY), (uint32_t)((i - 1) & 1), 2);
          tc_fence_after();
          if (__any_sync(0xffffffffu, changed)) {
            // rescale this warp's 32 rows of the output accumulator
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
              uint32_t o[32];
              const uint32_t o_addr = lane_base + 256u + (uint32_t)(cc * 32);
              CASCADE_TMEM_LD32(o_addr, o, 0);
              tmem_wait_ld();
#pragma unroll
              for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * (changed ? alpha : 1.f));
              CASCADE_TMEM_ST32(o_addr, o, 0);
            }
            tmem_wait_st();
          }
        }
        // P -> shared memory, K-major, 128-byte swizzle: row r, 16 chunks of 8 keys
#pragma unroll
        for (int ch = 0; ch < 16; ++ch) {
          uint4 val = make_uint4(pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2], pk[4 * ch + 3]);
          *reinterpret_cast<uint4*>(smem + kOffP + tile_offset(r, ch)) = val;
        }
        fence_proxy_async();
        tc_fence_before();
        mbar_arrive(bar(P_FULL));
      }
    }
    const int n_tiles = i;
    // ---- epilogue
    float o_scale = 0.f, m_out = -INFINITY, l_out = 0.f;
    if (n_tiles > 0) {
      wait_bar(wc, bar(P_EMPTY), (uint32_t)((n_tiles - 1) & 1), 3);
      tc_fence_after();
      if (l_run > 0.f) {
        o_scale = 1.f / l_run;
        l_out = l_run * ex2(m_run - m_true);  // sum relative to the exact max
        m_out = m_true * 0.6931471805599453f;   // natural-log units
      }
    }
    __nv_bfloat16* dst = nullptr;
    if (row_ok) {
      if (p.fused) {
        const int tok = __ldg(q_idx + row0 + r);
        dst = static_cast<__nv_bfloat16*>(p.o_out) + (int64_t)b * p.os.batch + (int64_t)tok * p.os.token +
              (int64_t)h * p.os.head;
        if (p.lse_out)
          p.lse_out[((int64_t)b * pl.n_q + tok) * p.H + h] = l_out > 0.f ? m_out + logf(l_out) : -INFINITY;
      } else {
        const int64_t stat = (((int64_t)b * P + part) * pl.n_q + (row0 + r)) * p.H + h;
        dst = static_cast<__nv_bfloat16*>(p.o_part) + stat * kD;
        p.m_part[stat] = m_out;
        p.l_part[stat] = l_out;
      }
    }
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
      uint32_t o[32];
      if (n_tiles > 0) {
        CASCADE_TMEM_LD32(lane_base + 256u + (uint32_t)(cc * 32), o, 0);
        tmem_wait_ld();
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) o[j] = 0u;
      }
      if (row_ok) {
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          uint4 val;
          val.x = pack_bf16x2(__uint_as_float(o[j]) * o_scale, __uint_as_float(o[j + 1]) * o_scale);
          val.y = pack_bf16x2(__uint_as_float(o[j + 2]) * o_scale, __uint_as_float(o[j + 3]) * o_scale);
          val.z = pack_bf16x2(__uint_as_float(o[j + 4]) * o_scale, __uint_as_float(o[j + 5]) * o_scale);
          val.w = pack_bf16x2(__uint_as_float(o[j + 6]) * o_scale, __uint_as_float(o[j + 7]) * o_scale);
          *reinterpret_cast<uint4*>(dst + cc * 32 + j) = val;
        }
      }
    }
    tc_fence_before();
  } else if (warp == 4) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = make_idesc(128, 128, 0, 0);
      constexpr uint32_t idesc_pv = make_idesc(128, 128, 0, 1);
      const uint32_t q_s = smem_base + kOffQ, p_s = smem_base + kOffP;
      int n_tiles = 0;
      for (int kk = k_begin; kk < k_end; ++kk) n_tiles += (__ldg(vis_last + kk) + kTile - 1) / kTile;
      auto issue_pv = [&](int j) {
        const int s = j % kStages;
        wait_bar(wc, bar(V_FULL + s), (uint32_t)((j / kStages) & 1), 4);
        wait_bar(wc, bar(P_FULL), (uint32_t)(j & 1), 5);
        tc_fence_after();
        const uint32_t v_s = smem_base + kOffV + s * kTileBytes;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          // A = P (K-major): 16 keys = 32 bytes along the row; B = V (MN-major): 16 keys = 16 rows of 128 bytes
          const uint64_t a = make_desc(p_s + (ks >> 2) * kHalfBytes + (ks & 3) * 32, 16, 1024);
          const uint64_t bd = make_desc(v_s + ks * 2048, kHalfBytes, 1024);
          mma_bf16(tmem + 256u, a, bd, idesc_pv, (j > 0 || ks > 0) ? 1u : 0u);
        }
        mma_commit(bar(V_EMPTY + s));
        mma_commit(bar(P_EMPTY));
      };
      if (n_tiles > 0) {
        wait_bar(wc, bar(Q_FULL), 0, 6);
        for (int i = 0; i < n_tiles; ++i) {
          const int s = i % kStages, sb = i & 1;
          wait_bar(wc, bar(K_FULL + s), (uint32_t)((i / kStages) & 1), 7);
          wait_bar(wc, bar(S_EMPTY + sb), (uint32_t)(((i >> 1) & 1) ^ 1), 8);
          tc_fence_after();
          const uint32_t k_s = smem_base + kOffK + s * kTileBytes;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
            mma_bf16(tmem + (uint32_t)(sb * 128), make_desc(q_s + off, 16, 1024), make_desc(k_s + off, 16, 1024),
                     idesc_qk, ks > 0 ? 1u : 0u);
          }
          mma_commit(bar(S_FULL + sb));
          mma_commit(bar(K_EMPTY + s));
          if (i > 0) issue_pv(i - 1);
        }
        issue_pv(n_tiles - 1);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ loaders (K: warps 5-6, V: warps 7-8)
    const bool is_k = warp < 7;
    const int t = tid - (is_k ? 160 : 224);  // 0..63
    const __nv_bfloat16* src = is_k ? static_cast<const __nv_bfloat16*>(p.k) + (int64_t)b * p.ks.batch +
                                          (int64_t)g * p.ks.head
                                    : static_cast<const __nv_bfloat16*>(p.v) + (int64_t)b * p.vs.batch +
                                          (int64_t)g * p.vs.head;
    const int64_t tstride = is_k ? p.ks.token : p.vs.token;
    const int full0 = is_k ? K_FULL : V_FULL, empty0 = is_k ? K_EMPTY : V_EMPTY;
    const uint32_t tiles_s = smem_base + (is_k ? kOffK : kOffV);
    int n_tiles = 0;
    for (int kk = k_begin; kk < k_end; ++kk) n_tiles += (__ldg(vis_last + kk) + kTile - 1) / kTile;
    if (n_tiles > 0) {
      int pending = -1;  // barrier to signal once the previously committed group has landed
      if (is_k) {
        const __nv_bfloat16* qsrc = static_cast<const __nv_bfloat16*>(p.q) + (int64_t)b * p.qs.batch +
                                    (int64_t)h * p.qs.head;
        gather_tile(smem_base + kOffQ, qsrc, p.qs.token, q_idx + row0, nrows, t, 64);
        cp_async_commit();
        pending = Q_FULL;
      }
      int i = 0;
      for (int kk = k_begin; kk < k_end; ++kk) {
        const int need = __ldg(vis_last + kk);
        const int32_t* idx = kv_idx + __ldg(kv_off + kk);
        for (int t0 = 0; t0 < need; t0 += kTile, ++i) {
          const int s = i % kStages;
          wait_bar(wc, bar(empty0 + s), (uint32_t)(((i / kStages) & 1) ^ 1), 9);
          gather_tile(tiles_s + s * kTileBytes, src, tstride, idx + t0, min(kTile, need - t0), t, 64);
          cp_async_commit();
          if (pending >= 0) {
            cp_async_wait<1>();  // everything but the group just committed has landed
            fence_proxy_async();
            mbar_arrive(bar(pending));
          }
          pending = full0 + s;
        }
      }
      cp_async_wait<0>();
      fence_proxy_async();
      if (pending >= 0) mbar_arrive(bar(pending));
    }
  }
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

}  // namespace tc

cudaError_t launch_attn_tc(const AttnParams& p, cudaStream_t stream) {
  cudaError_t e = cudaFuncSetAttribute(tc::attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       tc::kSmemBytes);
  if (e != cudaSuccess) return e;
  const int n_parts = p.fused ? 1 : p.plan.n_kv_shards;
  dim3 grid(p.plan.n_qtiles128, p.H, p.batch * n_parts);
  tc::attn_tc_kernel<<<grid, tc::kThreads, tc::kSmemBytes, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace cascade
