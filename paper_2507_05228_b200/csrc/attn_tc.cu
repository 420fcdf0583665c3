// Attention-pass on the 5th-generation tensor cores (tcgen05 + TMEM) for bf16, head_dim 128.
//
// Work decomposition.  The M dimension of one MMA tile (128 rows) is filled with (query slot, head) pairs: the
// Gp query heads that read the same KV head ("repeat_kv", Algorithm 3 lines 1-2) are stacked next to each other,
// so a tile covers only 128 / Gp consecutive slots of one query shard.  Under token sharding the rows of a shard
// are spread over the whole sequence, and the staircase between the shortest and the longest visible prefix of a
// tile is wasted tensor work; stacking heads shrinks that staircase by Gp.
// One CTA owns two such sub-tiles (the next 128 / Gp slots of the same shard, same heads), which share every K/V
// tile, and either one KV shard (partials: Algorithm 3 for the pair) or all KV shards one after another (fused:
// the carry n, w, o of Algorithm 4 is the running max / sum / output of the streaming softmax).
// Each shard's visible prefix is walked in tiles of at most 128 keys; the last tile of a prefix is narrowed to a
// multiple of 32 keys.
//
// Warp roles (12 warps):
//   0-3   softmax of sub-tile 0, 4-7 softmax of sub-tile 1: thread = MMA row = TMEM lane.  Reads the logits S with
//         tcgen05.ld, applies the shard mask (the row sees the first vis[slot][k] keys of the shard), keeps the running
//         max / sum, writes the probabilities P as bf16 back into the TMEM columns of S, rescales the output
//         accumulator in TMEM when the running max moved by more than 2^8, and runs the epilogue.
//   8     MMA issuer (one lane): S_s = Q_s K^T (operands in shared memory) and O_s += P_s V (P from TMEM),
//         issued as PV_0(i), QK_0(i+1), PV_1(i), QK_1(i+1) so that the tensor pipe works on one sub-tile while the
//         other is in its softmax.  QK_s(i+1) overwrites the columns PV_s(i) reads P from; MMAs execute in issue
//         order, which makes that safe without a barrier.
//   9-11  loaders: index-mapped gather of 256-byte rows with 16-byte cp.async into the 128-byte-swizzled layout
//         the MMA descriptors expect; warp 9 streams the K tiles, warps 10 and 11 the even and odd V tiles.
// Every mbarrier wait is bounded: on expiry the CTA raises a flag, records a code in the plan's status word
// and drains without waiting again.
#include "cascade_internal.cuh"

namespace cascade {
namespace tc {

constexpr int kThreads = 384;
constexpr int kM = 128;                  // MMA rows per sub-tile
constexpr int kNMax = 128;               // keys per KV tile (upper bound)
constexpr int kD = 128;                  // head_dim
constexpr int kTileBytes = kM * kD * 2;  // 32 KiB, laid out [2 halves][128 rows][128 bytes]
constexpr int kHalfBytes = kTileBytes / 2;
constexpr int kKStages = 3;
constexpr int kVStages = 2;
constexpr uint32_t kTmemCols = 512;       // S0 | S1 | O0 | O1, 128 columns each; P_s aliases the start of S_s
constexpr float kRescaleThreshold = 8.f;  // log2 units
constexpr int kRegsSoftmax = 216;
constexpr int kRegsOther = 72;

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + 2 * kTileBytes;
constexpr int kOffV = kOffK + kKStages * kTileBytes;
constexpr int kOffBar = kOffV + kVStages * kTileBytes;
constexpr int kNumBars = 24;
constexpr int kOffMisc = kOffBar + kNumBars * 8;
constexpr int kSmemBytes = kOffMisc + 64 + 1024;  // + alignment slack
static_assert(kSmemBytes <= 232448, "exceeds the 227 KiB a CTA may use");

enum Bar {
  Q_FULL = 0,                     // [2]
  K_FULL = 2,                     // [kKStages]
  K_EMPTY = K_FULL + kKStages,    // [kKStages]
  V_FULL = K_EMPTY + kKStages,    // [kVStages]
  V_EMPTY = V_FULL + kVStages,    // [kVStages]
  S_FULL = V_EMPTY + kVStages,    // [2]
  P_FULL = S_FULL + 2,            // [2]
  O_FULL = P_FULL + 2             // [1]
};
static_assert(O_FULL + 1 <= kNumBars, "barrier table too small");

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
  volatile int* progress;    // shared memory, one word per warp: 8 * tile + step, for the timeout report
  int32_t* status;           // global: [0] code, [1..3] block index, [4] tile of the waiter, [8..19] progress words
};

// Bounded wait: gives up after ~2 s, raises the CTA's abort flag and records `code`.
__device__ __forceinline__ bool wait_bar(const WaitCtx& c, uint32_t bar, uint32_t parity, int code, int tile = 0) {
  if (*c.abort_flag) return false;
  if (mbar_try_wait(bar, parity)) return true;
  uint64_t t0 = 0;
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 1023u) == 0) {
      if (*c.abort_flag || *reinterpret_cast<volatile int32_t*>(c.status) != 0) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      if (now - t0 > 2000000000ull) {
        *c.abort_flag = 1;
        if (atomicCAS(c.status, 0, code) == 0) {  // first CTA to give up: leave a report
          c.status[1] = (int32_t)blockIdx.x;
          c.status[2] = (int32_t)blockIdx.y;
          c.status[3] = (int32_t)blockIdx.z;
          c.status[4] = tile;
          for (int w = 0; w < kThreads / 32; ++w) c.status[8 + w] = c.progress[w];
        }
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
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

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]; A is 128 lanes x 8 columns, each column holding two consecutive bf16 along K
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
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

#define CASCADE_TMEM_ST16(taddr, r)                                                                            \
  asm volatile(                                                                                                 \
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "                                                          \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"                                 \
      ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),      \
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(taddr)           \
      : "memory")

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {  // 2^x, MUFU; ex2(-inf) = +0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float y;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
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

// The CTA's sequence of KV tiles: shard by shard, each shard's visible prefix (as seen by the CTA's last row, which
// has the longest one) in pieces of at most 128 keys.  Every role walks the same sequence.
struct TileWalk {
  const int32_t* need_of;  // vis[last row of the CTA][*]
  int k_end, kk, t0, need;
  __device__ __forceinline__ void seek() {
    t0 = 0;
    need = 0;
    while (kk < k_end) {
      need = __ldg(need_of + kk);
      if (need > 0) break;
      ++kk;
    }
  }
  __device__ __forceinline__ void start(const int32_t* need_of_, int k_begin, int k_end_) {
    need_of = need_of_;
    k_end = k_end_;
    kk = k_begin;
    seek();
  }
  __device__ __forceinline__ bool done() const { return kk >= k_end; }
  __device__ __forceinline__ int keys() const { return min(kNMax, need - t0); }  // real keys in this tile
  __device__ __forceinline__ int n() const { return (keys() + 31) & ~31; }       // MMA width: multiple of 32
  __device__ __forceinline__ void next() {
    t0 += kNMax;
    if (t0 >= need) {
      ++kk;
      seek();
    }
  }
};

// One warp gathers rows [0, n_rows) of a tile (n_rows a multiple of 32).  tok_of(row) returns the source token of the
// row or -1 for a zero-filled row; src_of(row, tok) returns the address of the row's 256 bytes.
template <typename TokOf, typename SrcOf>
__device__ __forceinline__ void gather_rows(uint32_t tile_saddr, int n_rows, int lane, TokOf tok_of, SrcOf src_of) {
  const int chunk = lane & 15, sub = lane >> 4;
  for (int r0 = 0; r0 < n_rows; r0 += 32) {
    const int my_tok = tok_of(r0 + lane);  // one coalesced index load per 32 rows
#pragma unroll
    for (int pp = 0; pp < 16; ++pp) {
      const int row = r0 + 2 * pp + sub;
      const int tok = __shfl_sync(0xffffffffu, my_tok, 2 * pp + sub);
      const bool ok = tok >= 0;
      cp_async16(tile_saddr + tile_offset(row, chunk), src_of(row, ok ? tok : 0) + chunk * 8, ok ? 16u : 0u);
    }
  }
}

__global__ void __launch_bounds__(kThreads, 1) attn_tc_kernel(AttnParams p, int lg) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar0 = smem_base + kOffBar;
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffMisc + 4);
  volatile int* progress = reinterpret_cast<volatile int*>(smem + kOffMisc + 8);  // [12]

  // lg = log2(Gp): Gp heads stacked per tile, R = 128 / Gp slots per sub-tile, 2 R slots per CTA
  const int Gp = 1 << lg, R = kM >> lg;
  const PlanDev& pl = p.plan;
  const int P = pl.n_kv_shards;
  const int n_parts = p.fused ? 1 : P;
  const int b = blockIdx.z / n_parts;
  const int part = blockIdx.z % n_parts;
  const int map = pl.n_maps == 1 ? 0 : b;
  const int h0 = blockIdx.y * Gp;  // first of the Gp stacked heads
  const int g = h0 / p.G;          // their KV head
  const int ts = 3 - lg;           // tile list of 2 R = 256 >> lg slots
  const int4 qt = pl.qtiles[ts][(size_t)map * pl.n_qtiles[ts] + blockIdx.x];
  const int row0 = qt.x, nrows = qt.y;
  if (nrows == 0) return;  // padding entry (uniform for the CTA)
  if (*reinterpret_cast<volatile int32_t*>(pl.status) != 0) return;  // an earlier CTA gave up: do not pile on
  const int n_sub = nrows > R ? 2 : 1;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int32_t* q_idx = pl.q_idx + (size_t)map * pl.n_q;
  const int32_t* kv_idx = pl.kv_idx + (size_t)map * pl.n_kv;
  const int32_t* kv_off = pl.kv_off + (size_t)map * (P + 1);
  const int32_t* vis = pl.vis + (size_t)map * pl.n_q * P;
  const int32_t* vis_last = vis + (size_t)(row0 + nrows - 1) * P;  // longest prefix of the CTA (rows ascend)
  const int k_begin = p.fused ? 0 : part, k_end = p.fused ? P : part + 1;
  WaitCtx wc{abort_flag, progress, pl.status};
  auto note = [&](int v) {
    if (lane == 0) progress[warp] = v;
  };

  if (tid == 0) {
    mbar_init(bar(Q_FULL), 32);
    mbar_init(bar(Q_FULL + 1), 32);
    for (int s = 0; s < kKStages; ++s) {
      mbar_init(bar(K_FULL + s), 32);
      mbar_init(bar(K_EMPTY + s), 1);
    }
    for (int s = 0; s < kVStages; ++s) {
      mbar_init(bar(V_FULL + s), 32);
      mbar_init(bar(V_EMPTY + s), 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar(S_FULL + s), 1);
      mbar_init(bar(P_FULL + s), 128);
    }
    mbar_init(bar(O_FULL), 1);
    *abort_flag = 0;
    for (int w = 0; w < kThreads / 32; ++w) progress[w] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
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

  if (warp < 8) {
    // ------------------------------------------------------------------ softmax + epilogue
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
    const int s = warp >> 2;  // sub-tile
    if (s < n_sub) {
      const int m = tid & 127;  // MMA row = TMEM lane
      const int sub_row0 = row0 + s * R;
      const int sub_nrows = min(R, nrows - s * R);
      const int slot_local = m >> lg;
      const bool row_ok = slot_local < sub_nrows;
      const int slot = sub_row0 + (row_ok ? slot_local : 0);
      const int head = h0 + (m & (Gp - 1));
      const int32_t* vis_row = vis + (size_t)slot * P;
      const int32_t* vis_first = vis + (size_t)sub_row0 * P;  // shortest prefix of the sub-tile
      const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
      const uint32_t s_addr = lane_base + (uint32_t)(s * 128);
      const uint32_t o_addr = lane_base + 256u + (uint32_t)(s * 128);
      const float c = p.scale * 1.4426950408889634f;  // logits are kept in log2 units: x = s * scale * log2(e)
      float m_run = -INFINITY;   // reference max the accumulators are scaled by (may lag by < 2^8)
      float m_true = -INFINITY;  // exact running max
      float l_run = 0.f;
      int my_vis = 0, full_upto = 0;
      int i = 0;  // KV tile counter
      TileWalk w;
      for (w.start(vis_last, k_begin, k_end); !w.done(); w.next(), ++i) {
        if (w.t0 == 0) {  // entered a new shard
          my_vis = row_ok ? __ldg(vis_row + w.kk) : 0;
          full_upto = __ldg(vis_first + w.kk);
        }
        const int n = w.n();
        const int nch = n >> 5;
        note(8 * i + 1);
        wait_bar(wc, bar(S_FULL + s), (uint32_t)(i & 1), 1, i);
        tc_fence_after();
        uint32_t sr[128];
        CASCADE_TMEM_LD32(s_addr, sr, 0);
        if (nch > 1) CASCADE_TMEM_LD32(s_addr + 32, sr, 32);
        if (nch > 2) CASCADE_TMEM_LD32(s_addr + 64, sr, 64);
        if (nch > 3) CASCADE_TMEM_LD32(s_addr + 96, sr, 96);
        tmem_wait_ld();
        // mask (only tiles that reach past the shortest prefix of the sub-tile need it) and tile max
        float tmax;
        if (n == kNMax && w.t0 + n <= full_upto) {  // every valid row of the sub-tile sees all 128 keys
          float mx[4];
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            mx[q4] = __uint_as_float(sr[32 * q4]);
#pragma unroll
            for (int j = 1; j < 31; j += 2)
              mx[q4] = fmax3(mx[q4], __uint_as_float(sr[32 * q4 + j]), __uint_as_float(sr[32 * q4 + j + 1]));
            mx[q4] = fmaxf(mx[q4], __uint_as_float(sr[32 * q4 + 31]));
          }
          tmax = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
        } else {
          const int lim = my_vis - w.t0;  // columns [0, lim) are visible to this row; lim <= keys <= n
          tmax = -INFINITY;
#pragma unroll
          for (int j = 0; j < 128; ++j) {
            if (j >= lim) sr[j] = 0xff800000u;  // -inf (also covers the columns that were never loaded)
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
        float psum0 = 0.f, psum1 = 0.f;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          if (ch < nch) {  // warp-uniform
            uint32_t pk[16];
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              const float p0 = ex2(fmaf(__uint_as_float(sr[32 * ch + j]), c, neg_m));
              const float p1 = ex2(fmaf(__uint_as_float(sr[32 * ch + j + 1]), c, neg_m));
              psum0 += p0;
              psum1 += p1;
              pk[j >> 1] = pack_bf16x2(p0, p1);
            }
            // P as the A operand of the PV product: lane = row, column kk holds keys 2 kk and 2 kk + 1
            CASCADE_TMEM_ST16(s_addr + (uint32_t)(16 * ch), pk);
          }
        }
        l_run = l_run * alpha + (psum0 + psum1);
        // S_FULL(i) was committed after PV(i-1), so the output accumulator is quiescent until this thread's
        // arrival on P_FULL(i) below
        if (i > 0 && __any_sync(0xffffffffu, changed)) {
          // rescale this warp's 32 rows of the output accumulator
          const float f = changed ? alpha : 1.f;
#pragma unroll
          for (int cc = 0; cc < 4; ++cc) {
            uint32_t o[32];
            CASCADE_TMEM_LD32(o_addr + (uint32_t)(cc * 32), o, 0);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * f);
            CASCADE_TMEM_ST32(o_addr + (uint32_t)(cc * 32), o, 0);
          }
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(P_FULL + s));
        note(8 * i + 2);
      }
      const int n_tiles = i;
      note(8 * i + 3);
      // ---- epilogue
      float o_scale = 0.f, m_out = -INFINITY, l_out = 0.f;
      if (n_tiles > 0) {
        wait_bar(wc, bar(O_FULL), 0u, 3, n_tiles);
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
          const int tok = __ldg(q_idx + slot);
          dst = static_cast<__nv_bfloat16*>(p.o_out) + (int64_t)b * p.os.batch + (int64_t)tok * p.os.token +
                (int64_t)head * p.os.head;
          if (p.lse_out)
            p.lse_out[((int64_t)b * pl.n_q + tok) * p.H + head] = l_out > 0.f ? m_out + logf(l_out) : -INFINITY;
        } else {
          const int64_t stat = (((int64_t)b * P + part) * pl.n_q + slot) * p.H + head;
          dst = static_cast<__nv_bfloat16*>(p.o_part) + stat * kD;
          p.m_part[stat] = m_out;
          p.l_part[stat] = l_out;
        }
      }
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t o[32];
        if (n_tiles > 0) {
          CASCADE_TMEM_LD32(o_addr + (uint32_t)(cc * 32), o, 0);
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
    }
  } else {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
    if (warp == 8) {
      // ---------------------------------------------------------------- MMA issuer
      if (lane == 0) {
        constexpr uint32_t idesc_pv = make_idesc(kM, kD, 0, 1);
        const uint32_t q_s = smem_base + kOffQ;
        TileWalk w;
        w.start(vis_last, k_begin, k_end);
        if (!w.done()) {
          auto issue_qk = [&](int s, int i, int n) {  // S_s = Q_s K(i)^T, n keys wide
            const uint32_t k_s = smem_base + kOffK + (i % kKStages) * kTileBytes;
            const uint32_t idesc_qk = make_idesc(kM, n, 0, 0);
#pragma unroll
            for (int ks = 0; ks < kD / 16; ++ks) {
              const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
              mma_ss(tmem + (uint32_t)(s * 128), make_desc(q_s + s * kTileBytes + off, 16, 1024),
                     make_desc(k_s + off, 16, 1024), idesc_qk, ks > 0 ? 1u : 0u);
            }
            mma_commit(bar(S_FULL + s));
          };
          auto issue_pv = [&](int s, int i, int n) {  // O_s (+)= P_s V(i) over n keys
            const uint32_t v_s = smem_base + kOffV + (i % kVStages) * kTileBytes;
            const int ksteps = n >> 4;
            for (int ks = 0; ks < ksteps; ++ks) {
              // A = P from TMEM: 16 keys = 8 columns; B = V (MN-major): 16 keys = 16 rows of 128 bytes
              mma_ts(tmem + 256u + (uint32_t)(s * 128), tmem + (uint32_t)(s * 128 + ks * 8),
                     make_desc(v_s + ks * 2048, kHalfBytes, 1024), idesc_pv, (i > 0 || ks > 0) ? 1u : 0u);
            }
          };
          int n_cur = w.n();
          wait_bar(wc, bar(K_FULL), 0u, 7);
          for (int s = 0; s < n_sub; ++s) {
            wait_bar(wc, bar(Q_FULL + s), 0u, 6);
            tc_fence_after();
            issue_qk(s, 0, n_cur);
          }
          mma_commit(bar(K_EMPTY));
          w.next();
          for (int i = 0;; ++i) {
            const bool has_next = !w.done();
            const int n_next = has_next ? w.n() : 0;
            progress[warp] = 8 * i + 1;
            wait_bar(wc, bar(V_FULL + i % kVStages), (uint32_t)((i / kVStages) & 1), 4, i);
            for (int s = 0; s < n_sub; ++s) {
              progress[warp] = 8 * i + 2 + s;
              wait_bar(wc, bar(P_FULL + s), (uint32_t)(i & 1), 5, i);
              tc_fence_after();
              issue_pv(s, i, n_cur);
              if (s == n_sub - 1) mma_commit(bar(V_EMPTY + i % kVStages));
              if (has_next) {
                if (s == 0) {
                  progress[warp] = 8 * i + 4;
                  wait_bar(wc, bar(K_FULL + (i + 1) % kKStages), (uint32_t)(((i + 1) / kKStages) & 1), 7, i);
                  tc_fence_after();
                }
                issue_qk(s, i + 1, n_next);
                if (s == n_sub - 1) mma_commit(bar(K_EMPTY + (i + 1) % kKStages));
              }
            }
            if (!has_next) break;
            n_cur = n_next;
            w.next();
          }
          mma_commit(bar(O_FULL));
          progress[warp] = 7;
        }
      }
      __syncwarp();
    } else {
      // ---------------------------------------------------------------- loaders
      // Every barrier is served by one warp only, in tile order: a phase-parity wait cannot tell "one phase behind"
      // from "one phase ahead", so a warp must never skip a use of a stage.
      //   warp 9: all K tiles, two gathers in flight (K(i) is announced once K(i+1) has been issued)
      //   warp 10: Q_0, then V(0), V(2), ...;  warp 11: Q_1, then V(1), V(3), ...   (V stage = tile parity)
      const int lw = warp - 9;
      const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(p.k) + (int64_t)b * p.ks.batch + (int64_t)g * p.ks.head;
      const __nv_bfloat16* vb = static_cast<const __nv_bfloat16*>(p.v) + (int64_t)b * p.vs.batch + (int64_t)g * p.vs.head;
      const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(p.q) + (int64_t)b * p.qs.batch + (int64_t)h0 * p.qs.head;
      TileWalk w;
      w.start(vis_last, k_begin, k_end);
      if (!w.done()) {
        if (lw >= 1 && lw - 1 < n_sub) {  // query sub-tile (row m = slot m / Gp, head m % Gp)
          const int s = lw - 1;
          const int sub_row0 = row0 + s * R;
          const int sub_nrows = min(R, nrows - s * R);
          gather_rows(
              smem_base + kOffQ + s * kTileBytes, kM, lane,
              [&](int row) { return (row >> lg) < sub_nrows ? __ldg(q_idx + sub_row0 + (row >> lg)) : -1; },
              [&](int row, int tok) { return qb + (int64_t)tok * p.qs.token + (int64_t)(row & (Gp - 1)) * p.qs.head; });
          cp_async_wait_all();
          fence_proxy_async();
          mbar_arrive(bar(Q_FULL + s));
        }
        int i = 0;
        int announced = -1;  // K stage whose gather has been issued but not yet announced
        for (; !w.done(); w.next(), ++i) {
          const int keys = w.keys(), n = w.n();
          const int32_t* idx = kv_idx + __ldg(kv_off + w.kk) + w.t0;
          auto tok_of = [&](int row) { return row < keys ? __ldg(idx + row) : -1; };
          if (lw == 0) {
            const int st = i % kKStages;
            note(8 * i + 1);
            wait_bar(wc, bar(K_EMPTY + st), (uint32_t)(((i / kKStages) & 1) ^ 1), 9, i);
            gather_rows(smem_base + kOffK + st * kTileBytes, n, lane, tok_of,
                        [&](int, int tok) { return kb + (int64_t)tok * p.ks.token; });
            cp_async_commit();
            if (announced >= 0) {
              cp_async_wait<1>();  // everything but the gather just issued has landed
              fence_proxy_async();
              mbar_arrive(bar(K_FULL + announced));
            }
            announced = st;
            note(8 * i + 2);
          } else if ((i & 1) == lw - 1) {
            static_assert(kVStages == 2, "V stage = tile parity = loader warp");
            const int st = i & 1;
            note(8 * i + 3);
            wait_bar(wc, bar(V_EMPTY + st), (uint32_t)(((i / kVStages) & 1) ^ 1), 10, i);
            gather_rows(smem_base + kOffV + st * kTileBytes, n, lane, tok_of,
                        [&](int, int tok) { return vb + (int64_t)tok * p.vs.token; });
            cp_async_wait_all();
            fence_proxy_async();
            mbar_arrive(bar(V_FULL + st));
            note(8 * i + 4);
          }
        }
        if (lw == 0 && announced >= 0) {
          cp_async_wait_all();
          fence_proxy_async();
          mbar_arrive(bar(K_FULL + announced));
        }
        note(8 * i + 7);
      }
      cp_async_wait_all();
    }
  }
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

}  // namespace tc

cudaError_t launch_attn_tc(const AttnParams& p, cudaStream_t stream) {
  cudaError_t e = cudaFuncSetAttribute(tc::attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       tc::kSmemBytes);
  if (e != cudaSuccess) return e;
  // stack as many of the G heads of a KV head into one MMA tile as divide G (at most 8)
  int lg = 0;
  while (lg < 3 && p.G % (2 << lg) == 0) ++lg;
  const int n_parts = p.fused ? 1 : p.plan.n_kv_shards;
  dim3 grid(p.plan.n_qtiles[3 - lg], p.H >> lg, p.batch * n_parts);
  tc::attn_tc_kernel<<<grid, tc::kThreads, tc::kSmemBytes, stream>>>(p, lg);
  count_launch();
  return cudaGetLastError();
}

}  // namespace cascade
