// Attention-pass on the 5th-generation tensor cores (tcgen05 + TMEM) for bf16, head_dim 128.
//
// Work decomposition.  The M dimension of one MMA tile (128 rows) is filled with (query slot, head) pairs: the
// Gp query heads that read the same KV head ("repeat_kv", the Attention-Pass algorithm) are stacked next to each other,
// so a tile covers only 128 / Gp consecutive slots of one query shard.  Under token sharding the rows of a shard
// are spread over the whole sequence, and the staircase between the shortest and the longest visible prefix of a
// tile is wasted tensor work; stacking heads shrinks that staircase by Gp.
// One CTA owns two such sub-tiles (the next 128 / Gp slots of the same shard, same heads), which share every K/V
// tile, and walks all KV shards one after another.  Fused route: the carry n, w, o of the Post-Pass algorithm is the
// running max / sum / output of the streaming softmax, and one output row is written at the end.  Partials (kWalk,
// the Attention-Pass algorithm for every pair of the query tile): a tile never mixes two shards, and at every shard
// boundary that shard's (u, m, l) is written out and the statistics and the accumulator start over.  (A CTA per
// (query tile, KV shard) pair is kept as a compile-time alternative; it pays the CTA set-up once per pair.)
// The KV shards are walked one after another; each shard's visible prefix (as seen by the CTA's last row, which has
// the longest one) is cut into chunks of 32 keys, and four consecutive chunks of that stream - possibly from
// different shards - form one MMA tile of 128 keys, so that only the last tile of a CTA is narrower.  (An MMA costs
// the same for 32 keys as for 128, and every tile costs one softmax round trip.)
//
// Warp roles (12 warps):
//   0-3   softmax of sub-tile 0, 4-7 softmax of sub-tile 1: thread = MMA row = TMEM lane.  Reads the logits S with
//         tcgen05.ld, applies the shard mask (the row sees the first vis[slot][k] keys of the shard), keeps the running
//         max / sum, writes the probabilities P as bf16 back into the TMEM columns of S, rescales the output
//         accumulator in TMEM when the running max moved by more than 2^8, and runs the epilogue: the scaled output
//         row goes through shared memory (the Q / K tiles are free by then) to the copy engine, one 256-byte bulk
//         copy per row.
//   8     MMA issuer: S_s = Q_s K^T (operands in shared memory) and O_s += P_s V (P from TMEM), issued as
//         PV_0(i), QK_0(i+1), PV_1(i), QK_1(i+1) so that the tensor pipe works on one sub-tile while the other is in
//         its softmax.  QK_s(i+1) overwrites the columns PV_s(i) reads P from; MMAs execute in issue order, which
//         makes that safe without a barrier.  The whole warp runs the loop and one elected lane issues, so that
//         descriptors and addresses stay warp-uniform.
//   9-10  loaders: TMA box loads, completion counted in bytes on an mbarrier, data written in the 128-byte-swizzled
//         layout the MMA descriptors expect.  Warp 9 streams the K tiles and warp 10 the V tiles from the
//         shard-major copies that the gather pass (gather.cu) wrote: the visible prefix of a shard is a
//         contiguous run of rows there, so a tile is two 16 KiB box loads.  An index-mapped gather straight from
//         the caller's tensors was far too slow for the K/V stream (measured: one 512-byte TMA row gather per ~36
//         cycles per SM; 16-byte cp.async: one 512-byte request per ~90 cycles per warp).  The two query
//         sub-tiles are gathered once per CTA by the softmax threads themselves (plain 16-byte loads).
//   11    builds the table of the shards the CTA sees anything of (what each role needs per shard, and the number of
//         chunks), then idles; it also keeps the register-reallocation groups of four warps whole.
// The grid is launched as a programmatic dependent of the gather grid: everything up to the loaders' first TMA load
// may run while the gather is still writing the shard-major copies (the loaders wait with griddepcontrol.wait).
// Every mbarrier wait is bounded: on expiry the CTA raises a flag, records a code in the plan's status word
// and drains without waiting again.
#include <cuda.h>

#include "cascade_internal.cuh"

#ifndef CASCADE_PARTIALS_WALK
#define CASCADE_PARTIALS_WALK 1
#endif

namespace cascade {
namespace tc {

constexpr int kThreads = 384;
constexpr int kM = 128;                  // MMA rows per sub-tile
constexpr int kNMax = 128;               // keys per KV tile (upper bound)
constexpr int kD = 128;                  // head_dim
constexpr int kTileBytes = kM * kD * 2;  // 32 KiB, laid out [2 halves][128 rows][128 bytes]
constexpr int kHalfBytes = kTileBytes / 2;
constexpr int kKStages = 2;  // (a third stage bought nothing)
constexpr int kVStages = 2;
constexpr uint32_t kTmemCols = 512;       // S0 | S1 | O0 | O1, 128 columns each; P_s aliases the start of S_s
constexpr float kRescaleThreshold = 8.f;  // log2 units
// setmaxnreg only redistributes the registers the CTA was launched with (168 per thread x 384 threads = 64512), and
// all four warps of an allocation group execute the same instruction: 8 warps x 32 x 216 + 4 warps x 32 x 72 = 64512.
// An increase that asks for more than the launch grant never returns.
constexpr int kRegsSoftmax = 216;
constexpr int kRegsOther = 72;
static_assert(8 * 32 * kRegsSoftmax + 4 * 32 * kRegsOther <= 168 * kThreads, "setmaxnreg would wait for registers forever");
constexpr int kChunk = 32;                // keys per chunk of the KV stream
constexpr int kChunkBytes = kChunk * 128; // one 64-column half of a chunk in a tile
constexpr int kMaxShards = 256;           // KV shards per CTA whose bookkeeping fits in shared memory
constexpr int kStageRowBytes = 272;       // output rows staged for the bulk copies: 256 bytes + 16 of padding

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + 2 * kTileBytes;
constexpr int kOffV = kOffK + kKStages * kTileBytes;
constexpr int kOffBar = kOffV + kVStages * kTileBytes;
static_assert(2 * kM * kStageRowBytes <= kOffV, "the output staging area must fit in the Q and K tiles");
constexpr int kNumBars = 24;
constexpr int kOffMisc = kOffBar + kNumBars * 8;   // tmem slot, abort flag, 12 progress words
constexpr int kOffShard = kOffMisc + 64;           // int32 [5][kMaxShards], see ShardTab
constexpr int kSmemBytes = kOffShard + 5 * kMaxShards * 4 + 1024;  // + alignment slack
static_assert(kSmemBytes <= 232448, "exceeds the 227 KiB a CTA may use");

enum Bar {
  Q_FULL = 0,                     // [2]
  K_FULL = 2,                     // [kKStages]
  K_EMPTY = K_FULL + kKStages,    // [kKStages]
  V_FULL = K_EMPTY + kKStages,    // [kVStages]
  V_EMPTY = V_FULL + kVStages,    // [kVStages]
  S_FULL = V_EMPTY + kVStages,    // [2]
  P_FULL = S_FULL + 2,            // [2]
  O_FULL = P_FULL + 2,            // [1]
  O_RDY = O_FULL + 1              // [2]  kWalk: the accumulator of a sub-tile holds a finished shard
};
static_assert(O_RDY + 2 <= kNumBars, "barrier table too small");

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
__device__ __forceinline__ bool elect_one() {  // true in exactly one lane of a converged warp
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
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

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// TMA box load: 32 rows x 64 elements of the 3-D tensor [matrix z][row y][column x] land as 32 rows of 128 bytes.
__device__ __forceinline__ void tma_tile3(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, as two 32-bit words.  Low word: start address >> 4 (bits 0-13),
// leading-dimension byte offset >> 4 (bits 16-29).  High word: stride-dimension byte offset >> 4 (bits 0-13),
// descriptor version 1 (bits 14-15), layout type 2 = SWIZZLE_128B (bits 29-31).  Stepping along K only changes the
// start address, so the issuing code adds small constants to a precomputed low word.
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr, uint32_t lbo_bytes) {
  return ((saddr & 0x3FFFFu) >> 4) | ((lbo_bytes >> 4) << 16);
}
__host__ __device__ constexpr uint32_t desc_hi(uint32_t sbo_bytes) { return (sbo_bytes >> 4) | (1u << 14) | (2u << 29); }
// Instruction descriptor for kind::f16: D fp32 (bits 4-5 = 1), A and B bf16 (bits 7-9, 10-12 = 1), operand
// majors (bit 15 A, bit 16 B; 0 = K-major, 1 = MN-major), N >> 3 at bits 17-22, M >> 4 at bits 24-28.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n, int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem]; both descriptors share the high word
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                       bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"((uint32_t)accumulate)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]; A is 128 lanes x 8 columns, each column holding two consecutive bf16 along K
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                       bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"((uint32_t)accumulate)
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
// two fp32 lanes in one 64-bit register (packed FMA / ADD halve the issue slots of the exponent loop)
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Bookkeeping of the shards of which the CTA sees anything ("active" shards, in walk order), in shared memory.
struct ShardTab {
  int32_t need[kMaxShards];    // visible prefix of the CTA's last row = keys of the shard that are walked
  int32_t first[2][kMaxShards];  // visible prefix of the first row of sub-tile 0 / 1: chunks below it need no mask
  int32_t slot0[kMaxShards];   // position of the shard's first key in the shard-major K/V copies
  int32_t kk[kMaxShards];      // shard id
};
// Cursor over the chunk stream: chunk c of active shard j.
struct ChunkCursor {
  int j, c, nc;  // nc = chunks of shard j
  __device__ __forceinline__ void start(const ShardTab* t, int n_act) {
    j = 0;
    c = 0;
    nc = n_act > 0 ? (t->need[0] + kChunk - 1) / kChunk : 0;
  }
  // moves to the next chunk; returns true if that entered a new shard
  __device__ __forceinline__ bool advance(const ShardTab* t, int n_act) {
    if (++c < nc) return false;
    ++j;
    c = 0;
    nc = j < n_act ? (t->need[j] + kChunk - 1) / kChunk : 0;
    return true;
  }
};

// Chunk count and shard-start flag of consecutive tiles, for the roles that do not walk the chunks themselves.
template <bool kWalk>
struct TileSeq {
  const ShardTab* t;
  int n_act, n_chunks, i, j, c, nc;
  __device__ __forceinline__ TileSeq(const ShardTab* tab, int n_active, int chunks)
      : t(tab), n_act(n_active), n_chunks(chunks), i(0), j(0), c(0) {
    nc = (kWalk && n_act > 0) ? (t->need[0] + kChunk - 1) / kChunk : 0;
  }
  // the next tile: its chunks; first = it opens a shard (kWalk) or the whole stream
  __device__ __forceinline__ int next(bool& first) {
    if constexpr (!kWalk) {
      first = i == 0;
      const int n = min(4, n_chunks - 4 * i);
      ++i;
      return n;
    } else {
      first = c == 0;
      const int n = min(4, nc - c);
      c += n;
      if (c >= nc) {
        ++j;
        c = 0;
        nc = j < n_act ? (t->need[j] + kChunk - 1) / kChunk : 0;
      }
      return n;
    }
  }
};

struct TmaArgs {
  CUtensorMap k, v;  // shard-major copies as [batch * kv_heads][n_kv][head_dim]
};

// kRope: the query rows are turned by the rotary embedding of their positions while they are staged (the key rows
// were turned by the gather pass), the Pre-Pass algorithm.
// kWalk: the partials of EVERY KV shard for one query tile in one CTA (the attention-pass of the nodes AttnNode_{j,1..beta}
// one after another): the shards are walked as in the fused mode, but a tile never mixes two shards, and at a shard
// boundary the softmax threads write that shard's (u, m, l) out and start over.  The query tile, the TMEM allocation,
// the barriers and the K/V pipelines are set up once per query tile instead of once per (query tile, KV shard).
template <bool kRope, bool kWalk>
__global__ void __launch_bounds__(kThreads, 1) attn_tc_kernel(const __grid_constant__ AttnParams p, int lg,
                                                              int tile_major,
                                                              const __grid_constant__ TmaArgs tma) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar0 = smem_base + kOffBar;
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffMisc + 4);
  volatile int* progress = reinterpret_cast<volatile int*>(smem + kOffMisc + 8);  // [12]
  ShardTab* tab = reinterpret_cast<ShardTab*>(smem + kOffShard);
  volatile int* stream_info = reinterpret_cast<volatile int*>(smem + kOffMisc + 56);  // [0] active shards, [1] chunks

  // lg = log2(Gp): Gp heads stacked per tile, R = 128 / Gp slots per sub-tile, 2 R slots per CTA
  const int Gp = 1 << lg, R = kM >> lg;
  const PlanDev& pl = p.plan;
  const int P = pl.n_kv_shards;
  const int n_parts = (p.fused || kWalk) ? 1 : P;
  // CTA index -> (query tile, batch, part, head group).  The tile lists are sorted by decreasing work.  With few CTAs
  // per SM the query tile is the slowest index, so that the heaviest CTAs of all heads and sequences start first and
  // the light ones fill the tail.  For a large problem the head group is slowest instead: the CTAs running at any
  // time then read the K/V of few KV heads, which keeps that stream in L2.
  const int n_hg = p.H >> lg;
  const int n_qt = pl.n_qtiles[3 - lg];
  int tile_idx, hg, bz;
  if (tile_major) {
    const int per_tile = n_hg * p.batch * n_parts;
    const int rem = blockIdx.x % per_tile;
    tile_idx = blockIdx.x / per_tile;
    hg = rem % n_hg;
    bz = rem / n_hg;
  } else {
    // the KV shards of one query tile (partials) are neighbours, so that its rows are read from HBM once and the
    // CTAs running at a time walk all shards of one KV head
    const int rem = blockIdx.x / (n_qt * n_parts);
    tile_idx = (blockIdx.x / n_parts) % n_qt;
    hg = rem % n_hg;
    bz = (rem / n_hg) * n_parts + blockIdx.x % n_parts;
  }
  const int b = bz / n_parts;
  const int part = bz % n_parts;
  const int map = pl.n_maps == 1 ? 0 : b;
  const int h0 = hg * Gp;  // first of the Gp stacked heads
  const int g = h0 / p.G;  // their KV head
  const int ts = 3 - lg;   // tile list of 2 R = 256 >> lg slots
  const int4 qt = pl.qtiles[ts][(size_t)map * pl.n_qtiles[ts] + tile_idx];
  const int row0 = qt.x, nrows = qt.y;
  if (nrows == 0) return;  // padding entry (uniform for the CTA)
  if (*reinterpret_cast<volatile int32_t*>(pl.status) != 0) return;  // an earlier CTA gave up: do not pile on
  const int n_sub = nrows > R ? 2 : 1;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int32_t* q_idx = pl.q_idx + (size_t)map * pl.n_q;
  const int32_t* kv_off = pl.kv_off + (size_t)map * (P + 1);
  const int32_t* vis = pl.vis + (size_t)map * pl.n_q * P;
  const int k_begin = (p.fused || kWalk) ? 0 : part, k_end = (p.fused || kWalk) ? P : part + 1;
  // Query sub-tiles (row r = slot r / Gp, head r % Gp): the 128 softmax threads of a sub-tile gather it from the
  // caller's tensor, 16 bytes per thread and row, half a warp per 256-byte row.  The loads are issued here, before the
  // set-up below, and land in shared memory (128-byte-swizzled [2][128][128 B] layout) after it.  Rows past the end
  // of the sub-tile repeat its last row (their results are discarded).
  uint4 qv[16];
  const int q_chunk = tid & 15;
  const float4* rope_row[kRope ? 8 : 1];  // this thread's slice of the table row of each of its query rows
  float4 cs[kRope ? 4 : 1][4];            // (cos, sin) of four rows: 8 pairs each
  if (warp < 8 && (warp >> 2) < n_sub) {
    const int s = warp >> 2;
    const int sub_row0 = row0 + s * R;
    const int sub_nrows = min(R, nrows - s * R);
    if constexpr (kRope) {
      // Rotary staging: a thread holds both halves of 8 rotation pairs of a row (columns 8 c .. and 64 + 8 c ..),
      // 8 threads per row, 8 rows per thread, and the (cos, sin) of the first four of its rows; the table rows of the
      // other four are fetched while those are turned.
      const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(p.q) + (int64_t)b * p.qs.batch + (tid & 7) * 8;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int r = (tid >> 3 & 15) + 16 * j;
        const int tok =
            (int)CASCADE_CHECKED((int64_t)__ldg(q_idx + sub_row0 + min(r >> lg, sub_nrows - 1)), pl.n_q, pl.status, 108);
        const __nv_bfloat16* row = qb + (int64_t)tok * p.qs.token + (int64_t)(h0 + (r & (Gp - 1))) * p.qs.head;
        qv[2 * j] = __ldg(reinterpret_cast<const uint4*>(row));
        qv[2 * j + 1] = __ldg(reinterpret_cast<const uint4*>(row + 64));
        rope_row[j] = reinterpret_cast<const float4*>(p.rope + (int64_t)(pl.q_pos_offset + tok) * 64 + (tid & 7) * 8);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) cs[j][e] = __ldg(rope_row[j] + e);
    } else {
      const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(p.q) + (int64_t)b * p.qs.batch + q_chunk * 8;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int r = (tid >> 4 & 7) + 8 * j;
        const int tok =
            (int)CASCADE_CHECKED((int64_t)__ldg(q_idx + sub_row0 + min(r >> lg, sub_nrows - 1)), pl.n_q, pl.status, 108);
        qv[j] = __ldg(reinterpret_cast<const uint4*>(qb + (int64_t)tok * p.qs.token +
                                                     (int64_t)(h0 + (r & (Gp - 1))) * p.qs.head));
      }
    }
  }
  if (warp == 11) {  // the warp without a role of its own
    // Compact the shards of which the CTA's last row (longest prefix; rows ascend) sees something, with what the
    // roles need per shard, and count the chunks of the stream.
    const int32_t* need_of = vis + (size_t)(row0 + nrows - 1) * P;
    const int32_t* first0 = vis + (size_t)row0 * P;
    const int32_t* first1 = vis + (size_t)(row0 + (n_sub - 1) * R) * P;
    int n_act = 0, n_chunks = 0;
    for (int base = k_begin; base < k_end; base += 32) {
      const int kk = base + lane;
      const int nd = kk < k_end ? __ldg(need_of + kk) : 0;
      const uint32_t act = __ballot_sync(0xffffffffu, nd > 0);
      if (nd > 0) {
        const int pos = n_act + __popc(act & ((1u << lane) - 1u));
        tab->need[pos] = nd;
        tab->first[0][pos] = __ldg(first0 + kk);
        tab->first[1][pos] = __ldg(first1 + kk);
        tab->slot0[pos] = __ldg(kv_off + kk);
        tab->kk[pos] = kk;
      }
      n_act += __popc(act);
      int ch = (nd + kChunk - 1) / kChunk;
      if (kWalk) ch = (ch + 3) >> 2;  // tiles of this shard: a tile does not continue into the next shard
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) ch += __shfl_xor_sync(0xffffffffu, ch, off);
      n_chunks += ch;
    }
    if (lane == 0) {
      stream_info[0] = n_act;
      stream_info[1] = n_chunks;
    }
  }
  WaitCtx wc{abort_flag, progress, pl.status};
  auto note = [&](int v) {
    if (lane == 0) progress[warp] = v;
  };

  if (tid == 0) {
    mbar_init(bar(Q_FULL), 128);  // every thread of the sub-tile's softmax group brings a share of the rows
    mbar_init(bar(Q_FULL + 1), 128);
    for (int s = 0; s < kKStages; ++s) {
      mbar_init(bar(K_FULL + s), 1);  // TMA: one arrival that announces the byte count, then the bytes
      mbar_init(bar(K_EMPTY + s), 1);
    }
    for (int s = 0; s < kVStages; ++s) {
      mbar_init(bar(V_FULL + s), 1);
      mbar_init(bar(V_EMPTY + s), 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar(S_FULL + s), 1);
      mbar_init(bar(P_FULL + s), 128);
    }
    mbar_init(bar(O_FULL), 1);
    mbar_init(bar(O_RDY), 1);
    mbar_init(bar(O_RDY + 1), 1);
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
  const int n_act = stream_info[0];                 // shards of which the CTA sees something
  const int n_chunks = stream_info[1];              // chunks of the KV stream (kWalk: tiles, counted per shard)
  // MMA tiles: four chunks each; only the last one is narrower, or with kWalk the last one of every shard
  const int n_tiles = kWalk ? n_chunks : (n_chunks + 3) >> 2;
  auto tile_chunks = [&](int i) { return min(4, n_chunks - 4 * i); };  // not with kWalk: see TileSeq

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
      const int32_t* vis_first = tab->first[s];  // shortest prefix of the sub-tile, per active shard
      const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
      const uint32_t s_addr = lane_base + (uint32_t)(s * 128);
      const uint32_t o_addr = lane_base + 256u + (uint32_t)(s * 128);
      const float c = p.scale * 1.4426950408889634f;  // logits are kept in log2 units: x = s * scale * log2(e)
      const uint64_t c2 = pack2(c, c);
      float m_run = -INFINITY;   // reference max the accumulators are scaled by (may lag by < 2^8)
      float m_true = -INFINITY;  // exact running max
      float l_run = 0.f;
      if (n_tiles > 0) {
if constexpr (kRope) {
          // q <- rotary_pos_emb(q, p): (lo, hi) = (x[i], x[i + 64]) -> (lo cos - hi sin, hi cos + lo sin) in fp32,
          // rounded once to bf16, then stored like the unrotated rows
          uint8_t* q_tile = smem + kOffQ + s * kTileBytes;
          const int c = tid & 7;
          auto turn_and_store = [&](int j, const float4 (&t)[4]) {
            __nv_bfloat162* lo = reinterpret_cast<__nv_bfloat162*>(&qv[2 * j]);
            __nv_bfloat162* hi = reinterpret_cast<__nv_bfloat162*>(&qv[2 * j + 1]);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 a = __bfloat1622float2(lo[e]), h = __bfloat1622float2(hi[e]);
              lo[e] = __floats2bfloat162_rn(a.x * t[e].x - h.x * t[e].y, a.y * t[e].z - h.y * t[e].w);
              hi[e] = __floats2bfloat162_rn(h.x * t[e].x + a.x * t[e].y, h.y * t[e].z + a.y * t[e].w);
            }
            const int r = (tid >> 3 & 15) + 16 * j;
            uint8_t* dst = q_tile + r * 128 + ((c ^ (r & 7)) << 4);
            *reinterpret_cast<uint4*>(dst) = qv[2 * j];
            *reinterpret_cast<uint4*>(dst + kHalfBytes) = qv[2 * j + 1];
          };
          float4 cs2[4][4];
#pragma unroll
          for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) cs2[j][e] = __ldg(rope_row[4 + j] + e);
#pragma unroll
          for (int j = 0; j < 4; ++j) turn_and_store(j, cs[j]);
#pragma unroll
          for (int j = 0; j < 4; ++j) turn_and_store(4 + j, cs2[j]);
        } else {
          uint8_t* q_tile = smem + kOffQ + s * kTileBytes + (q_chunk >> 3) * kHalfBytes;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int r = (tid >> 4 & 7) + 8 * j;
            *reinterpret_cast<uint4*>(q_tile + r * 128 + (((q_chunk & 7) ^ (r & 7)) << 4)) = qv[j];
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> tensor-core reads
        mbar_arrive(bar(Q_FULL + s));
      }
      // This row's prefix lengths in the current and the next three active shards (a tile spans at most four), fetched
      // as the stream moves on so that the loads are off the critical path.
      auto row_vis = [&](int j) { return (j < n_act && row_ok) ? __ldg(vis_row + tab->kk[j]) : 0; };
      int vq0 = row_vis(0), vq1 = row_vis(1), vq2 = row_vis(2), vq3 = row_vis(3);
      ChunkCursor cur;
      cur.start(tab, n_act);
      int kk_open = -1;  // kWalk: the shard whose partial is being accumulated
      int n_flushed = 0;  // kWalk: partials written so far
      const bool rows32 = (reinterpret_cast<uintptr_t>(p.o_part) & 31) == 0;  // partial rows are 256 bytes apart
      // kWalk: writes the finished partial of shard kk (this thread's row of u, and m, l) straight from TMEM and the
      // running statistics, then starts over.  The row goes out as sixteen 16-byte stores.
      auto flush_shard = [&](int kk) {
        float o_scale = 0.f, m_out = -INFINITY, l_out = 0.f;
        if (l_run > 0.f) {
          o_scale = 1.f / l_run;
          l_out = l_run * ex2(m_run - m_true);
          m_out = m_true * 0.6931471805599453f;
        }
        const int64_t stat = (((int64_t)b * P + kk) * pl.n_q + slot) * p.H + head;
        if (row_ok) {
          p.m_part[stat] = m_out;
          p.l_part[stat] = l_out;
        }
        __nv_bfloat16* dst0 = static_cast<__nv_bfloat16*>(p.o_part) + stat * kD;
        // 64 columns per round trip, then 32-byte stores: a row's 16-byte pieces would half-fill 32 sectors per store
        // instruction
#pragma unroll
        for (int half = 0; half < 2; ++half) {
        uint32_t o[64];
        CASCADE_TMEM_LD32(o_addr + (uint32_t)(half * 64), o, 0);
        CASCADE_TMEM_LD32(o_addr + (uint32_t)(half * 64 + 32), o, 32);
        tmem_wait_ld();
        if (row_ok) {
          __nv_bfloat16* dst = dst0 + half * 64;
#pragma unroll
          for (int j = 0; j < 64; j += 16) {
            uint32_t w[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
              w[e] = pack_bf16x2(__uint_as_float(o[j + 2 * e]) * o_scale, __uint_as_float(o[j + 2 * e + 1]) * o_scale);
            if (rows32) {
              asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + j), "r"(w[0]),
                           "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                           : "memory");
            } else {
              *reinterpret_cast<uint4*>(dst + j) = make_uint4(w[0], w[1], w[2], w[3]);
              *reinterpret_cast<uint4*>(dst + j + 8) = make_uint4(w[4], w[5], w[6], w[7]);
            }
          }
        }
        }
        m_run = -INFINITY;
        m_true = -INFINITY;
        l_run = 0.f;
      };
      for (int i = 0; i < n_tiles; ++i) {
        // kWalk: a tile holds chunks of one shard only; the cursor stands at the tile's first chunk
        const int nch = kWalk ? min(4, cur.nc - cur.c) : tile_chunks(i);
        const bool opens = kWalk ? cur.c == 0 : i == 0;  // first tile of a shard (kWalk) or of the stream
        const int kk_tile = kWalk ? tab->kk[cur.j] : 0;
        // Mask bookkeeping for the tile's four chunks, done before the wait so that it costs nothing: a chunk of shard
        // j starting at key t0 needs the mask only if it reaches past the shortest prefix of the sub-tile; this row
        // then sees its first lc = vis - t0 columns.  Chunks a narrow last tile does not have count as fully masked.
        int lc[4];
        uint32_t needm = 0;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          if (ch < nch) {  // warp-uniform
            const int t0 = cur.c * kChunk;
            if (t0 + kChunk > vis_first[cur.j]) needm |= 1u << ch;
            lc[ch] = vq0 - t0;
            if (cur.advance(tab, n_act)) {
              vq0 = vq1;
              vq1 = vq2;
              vq2 = vq3;
              vq3 = row_vis(cur.j + 3);
            }
          } else {
            needm |= 1u << ch;
            lc[ch] = 0;
          }
        }
        note(8 * i + 1);
        if constexpr (kWalk) {
          // The issuing warp commits O_RDY right after the last product of a shard, before it issues the logits of
          // this tile, so the previous shard's partial is written out while those logits are computed.  The first
          // product of this shard (which overwrites the accumulator) waits for this thread's arrival on P_FULL(i).
          if (opens) {
            if (i > 0) {
              wait_bar(wc, bar(O_RDY + s), (uint32_t)(n_flushed & 1), 2, i);
              tc_fence_after();
              flush_shard(kk_open);
              ++n_flushed;
            }
            kk_open = kk_tile;
          }
        }
        wait_bar(wc, bar(S_FULL + s), (uint32_t)(i & 1), 1, i);
        tc_fence_after();
        uint32_t sr[128];
        CASCADE_TMEM_LD32(s_addr, sr, 0);
        if (nch > 1) CASCADE_TMEM_LD32(s_addr + 32, sr, 32);
        if (nch > 2) CASCADE_TMEM_LD32(s_addr + 64, sr, 64);
        if (nch > 3) CASCADE_TMEM_LD32(s_addr + 96, sr, 96);
        tmem_wait_ld();
        // The mask is applied through a bit mask so that the compiler can move several bits at a time into predicates.
        if (needm != 0) {  // warp-uniform
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            if ((needm >> ch) & 1u) {  // warp-uniform
              const uint32_t mk = lc[ch] >= 32 ? 0xffffffffu : (lc[ch] <= 0 ? 0u : ((1u << lc[ch]) - 1u));
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (!((mk >> j) & 1u)) sr[32 * ch + j] = 0xff800000u;  // -inf
            }
          }
        }
        float mx[4];
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          mx[q4] = __uint_as_float(sr[32 * q4]);
#pragma unroll
          for (int j = 1; j < 31; j += 2)
            mx[q4] = fmax3(mx[q4], __uint_as_float(sr[32 * q4 + j]), __uint_as_float(sr[32 * q4 + j + 1]));
          mx[q4] = fmaxf(mx[q4], __uint_as_float(sr[32 * q4 + 31]));
        }
        const float smax = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));  // raw logit
        const float tmax = smax * c;
        m_true = fmaxf(m_true, tmax);
        float m_new = m_run;
        if (m_run == -INFINITY || m_true > m_run + kRescaleThreshold) m_new = m_true;
        const float alpha = (m_run == -INFINITY) ? 0.f : ex2(m_run - m_new);
        const bool changed = m_new != m_run;
        m_run = m_new;
        const float neg_m = (m_run == -INFINITY) ? 0.f : -m_run;
        const uint64_t neg_m2 = pack2(neg_m, neg_m);
        uint64_t psum2 = pack2(0.f, 0.f);
        auto exp_chunk = [&](int ch) {
          uint32_t pk[16];
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            float x0, x1;
            unpack2(ffma2(pack2(__uint_as_float(sr[32 * ch + j]), __uint_as_float(sr[32 * ch + j + 1])), c2, neg_m2), x0,
                    x1);
            const float p0 = ex2(x0), p1 = ex2(x1);
            psum2 = fadd2(psum2, pack2(p0, p1));
            pk[j >> 1] = pack_bf16x2(p0, p1);
          }
          // P as the A operand of the PV product: lane = row, column kk holds keys 2 kk and 2 kk + 1
          CASCADE_TMEM_ST16(s_addr + (uint32_t)(16 * ch), pk);
        };
        if (nch == 4) {
          // The full tile is one straight-line block, so that the scheduler can run the MUFU instructions of one chunk
          // (8 issue cycles each) under the FMA / convert / store work of its neighbours; with a branch per chunk the
          // two parts ran back to back (1600 cycles per tile instead of the ~1130 the MUFU unit needs).
          exp_chunk(0);
          exp_chunk(1);
          exp_chunk(2);
          exp_chunk(3);
        } else {
#pragma unroll
          for (int ch = 0; ch < 3; ++ch)
            if (ch < nch) exp_chunk(ch);  // warp-uniform
        }
        float psum0, psum1;
        unpack2(psum2, psum0, psum1);
        // The tensor core multiplies the weights after rounding them to bf16, while the sum above is taken before.
        // With the lagging reference max even the largest weight of a row has an arbitrary mantissa, so when one key
        // dominates a row its rounding error (up to 2^-9 relative) would go straight into O / l: 0.009 at |v| = 4.5.
        // The sum therefore takes the tile's largest weight as the tensor core sees it (same fma and ex2 as in the
        // loop above, so the same bits); the other weights' errors are small against l or average out.
        const float p_top = ex2(fmaf(smax, c, neg_m));
        const float p_top_seen = __uint_as_float(pack_bf16x2(0.f, p_top) & 0xffff0000u);
        l_run = l_run * alpha + ((psum0 + psum1) + (p_top_seen - p_top));
        // S_FULL(i) was committed after PV(i-1), so the output accumulator is quiescent until this thread's
        // arrival on P_FULL(i) below
        if (!opens && __any_sync(0xffffffffu, changed)) {
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
      note(8 * n_tiles + 3);
      // ---- epilogue
      // Where this row goes is looked up before the wait for the last product, which hides the load.
      __nv_bfloat16* dst = nullptr;
      int64_t stat = 0;
      if (row_ok) {
        if (p.fused) {
          const int tok = (int)CASCADE_CHECKED((int64_t)__ldg(q_idx + slot), pl.n_q, pl.status, 109);
          stat = ((int64_t)b * pl.n_q + tok) * p.H + head;
          dst = static_cast<__nv_bfloat16*>(p.o_out) + (int64_t)b * p.os.batch + (int64_t)tok * p.os.token +
                (int64_t)head * p.os.head;
        } else {
          // kWalk: the last shard the CTA saw anything of; its other shards were written on the way
          stat = (((int64_t)b * P + (kWalk ? max(kk_open, 0) : part)) * pl.n_q + slot) * p.H + head;
          dst = static_cast<__nv_bfloat16*>(p.o_part) + stat * kD;
        }
      }
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
      if (row_ok) {
        if (p.fused) {
          if (p.lse_out) p.lse_out[stat] = l_out > 0.f ? m_out + logf(l_out) : -INFINITY;
        } else {
          p.m_part[stat] = m_out;
          p.l_part[stat] = l_out;
        }
      }
      // Every product of the CTA has completed, so the Q / K tiles in shared memory are free: the thread stages its
      // 256-byte output row there (rows 272 bytes apart, which spreads a warp's 16-byte stores over all banks) and hands
      // it to the copy engine as one bulk copy, instead of writing 32-byte pieces of 32 different rows per instruction.
      uint8_t* stage = smem + kOffQ + (s * kM + m) * kStageRowBytes;
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
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          uint4 val;
          val.x = pack_bf16x2(__uint_as_float(o[j]) * o_scale, __uint_as_float(o[j + 1]) * o_scale);
          val.y = pack_bf16x2(__uint_as_float(o[j + 2]) * o_scale, __uint_as_float(o[j + 3]) * o_scale);
          val.z = pack_bf16x2(__uint_as_float(o[j + 4]) * o_scale, __uint_as_float(o[j + 5]) * o_scale);
          val.w = pack_bf16x2(__uint_as_float(o[j + 6]) * o_scale, __uint_as_float(o[j + 7]) * o_scale);
          *reinterpret_cast<uint4*>(stage + cc * 64 + j * 2) = val;
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // this thread's writes -> the copy engine's reads
      if (row_ok) {
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], 256;" ::"l"(dst), "r"(smem_u32(stage))
                     : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // the row has left shared memory
      }
      if constexpr (kWalk) {
        // the shards of which no row of the CTA sees anything were never walked: their partials are empty
        if (row_ok) {
          int a = 0;
          for (int k = 0; k < P; ++k) {
            if (a < n_act && tab->kk[a] == k) {
              ++a;
              continue;
            }
            if (n_act == 0 && k == 0) continue;  // written by the epilogue above
            const int64_t st2 = (((int64_t)b * P + k) * pl.n_q + slot) * p.H + head;
            p.m_part[st2] = -INFINITY;
            p.l_part[st2] = 0.f;
            uint4* row = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.o_part) + st2 * kD);
#pragma unroll
            for (int j = 0; j < 16; ++j) row[j] = make_uint4(0u, 0u, 0u, 0u);
          }
        }
      }
      tc_fence_before();
    }
  } else {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
    if (warp == 8) {
      // ---------------------------------------------------------------- MMA issuer
      // All 32 lanes run the loop (waits included) so that every address and descriptor is warp-uniform; the
      // tcgen05 instructions themselves are issued by one elected lane.
      const bool leader = elect_one();
      constexpr uint32_t idesc_pv = make_idesc(kM, kD, 0, 1);
      constexpr uint32_t hi_kmajor = desc_hi(1024);  // Q, K: 8-row groups 1024 bytes apart
      constexpr uint32_t hi_v = desc_hi(1024);       // V (MN-major): 8-key groups 1024 bytes apart
      const uint32_t q_lo0 = desc_lo(smem_base + kOffQ, 16);
      const uint32_t k_lo0 = desc_lo(smem_base + kOffK, 16);
      const uint32_t v_lo0 = desc_lo(smem_base + kOffV, kHalfBytes);  // the two 64-column halves of d
      if (n_tiles > 0) {
        auto issue_qk = [&](int s, int i, int n) {  // S_s = Q_s K(i)^T, n keys wide
          const uint32_t q_lo = q_lo0 + (uint32_t)(s * (kTileBytes >> 4));
          const uint32_t k_lo = k_lo0 + (uint32_t)((i % kKStages) * (kTileBytes >> 4));
          const uint32_t idesc_qk = make_idesc(kM, n, 0, 0);
          if (leader) {
#pragma unroll
            for (int ks = 0; ks < kD / 16; ++ks) {
              // 16 elements of head_dim = 32 bytes along the 128-byte row; elements 64.. live in the second half
              const uint32_t off = (uint32_t)(((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4);
              mma_ss(tmem + (uint32_t)(s * 128), q_lo + off, k_lo + off, hi_kmajor, idesc_qk, ks > 0);
            }
            mma_commit(bar(S_FULL + s));
          }
        };
        // O_s (+)= P_s V(i) over n keys; a tile that opens a shard (kWalk) or the stream starts the accumulator afresh
        auto issue_pv = [&](int s, int i, int n, bool opens) {
          const uint32_t v_lo = v_lo0 + (uint32_t)((i % kVStages) * (kTileBytes >> 4));
          const int ksteps = n >> 4;
          if (leader) {
#pragma unroll
            for (int ks = 0; ks < kNMax / 16; ++ks) {
              // A = P from TMEM: 16 keys = 8 columns; B = V (MN-major): 16 keys = 16 rows of 128 bytes
              if (ks < ksteps)
                mma_ts(tmem + 256u + (uint32_t)(s * 128), tmem + (uint32_t)(s * 128 + ks * 8),
                       v_lo + (uint32_t)(ks * (2048 >> 4)), hi_v, idesc_pv, !opens || ks > 0);
            }
          }
        };
        TileSeq<kWalk> seq(tab, n_act, n_chunks);
        bool opens_cur = true, opens_next = false;
        int n_cur = kChunk * seq.next(opens_cur), n_next = 0;
        wait_bar(wc, bar(K_FULL), 0u, 7);
        for (int s = 0; s < n_sub; ++s) {
          wait_bar(wc, bar(Q_FULL + s), 0u, 6);
          tc_fence_after();
          issue_qk(s, 0, n_cur);
        }
        if (leader) mma_commit(bar(K_EMPTY));
        for (int i = 0; i < n_tiles; ++i) {
          const bool has_next = i + 1 < n_tiles;
          if (i > 0) {
            n_cur = n_next;
            opens_cur = opens_next;
          }
          n_next = has_next ? kChunk * seq.next(opens_next) : 0;
          note(8 * i + 1);
          wait_bar(wc, bar(V_FULL + i % kVStages), (uint32_t)((i / kVStages) & 1), 4, i);
          for (int s = 0; s < n_sub; ++s) {
            note(8 * i + 2 + s);
            wait_bar(wc, bar(P_FULL + s), (uint32_t)(i & 1), 5, i);
            tc_fence_after();
            issue_pv(s, i, n_cur, opens_cur);
            if (kWalk && has_next && opens_next && leader) mma_commit(bar(O_RDY + s));
            if (s == n_sub - 1 && leader) mma_commit(bar(V_EMPTY + i % kVStages));
            if (has_next) {
              if (s == 0) {
                note(8 * i + 4);
                wait_bar(wc, bar(K_FULL + (i + 1) % kKStages), (uint32_t)(((i + 1) / kKStages) & 1), 7, i);
                tc_fence_after();
              }
              issue_qk(s, i + 1, n_next);
              if (s == n_sub - 1 && leader) mma_commit(bar(K_EMPTY + (i + 1) % kKStages));
            }
          }
        }
        if (leader) mma_commit(bar(O_FULL));
        note(7);
      }
      __syncwarp();
    } else {
      // ---------------------------------------------------------------- loaders
      // Every barrier is served by one warp only, in tile order: a phase-parity wait cannot tell "one phase behind"
      // from "one phase ahead", so a warp must never skip a use of a stage.
      //   warp 9: the K tiles, warp 10: the V tiles (warp 11 has no work).
      const int lw = warp - 9;
      if (n_tiles > 0 && lw < 2) {
        const bool is_k = lw == 0;
        const CUtensorMap* map = is_k ? &tma.k : &tma.v;
        const int z = b * p.Hkv + g;  // which [n_kv][head_dim] matrix of the shard-major copy
        const int n_stages = is_k ? kKStages : kVStages;
        const int full0 = is_k ? K_FULL : V_FULL, empty0 = is_k ? K_EMPTY : V_EMPTY;
        const uint32_t tiles_s = smem_base + (is_k ? kOffK : kOffV);
        const bool leader = elect_one();
        ChunkCursor cur;
        cur.start(tab, n_act);
        // The shard-major copies are written by the gather grid launched just before this one; when this grid was
        // launched as its programmatic dependent it may have started early, so wait here for that grid to complete
        // (a no-op otherwise).  Nothing else in this kernel reads what the gather grid writes.
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int i = 0; i < n_tiles; ++i) {
          const int nch = kWalk ? min(4, cur.nc - cur.c) : tile_chunks(i);
          const int st = i % n_stages;
          note(8 * i + 1);
          wait_bar(wc, bar(empty0 + st), (uint32_t)(((i / n_stages) & 1) ^ 1), is_k ? 9 : 10, i);
          const uint32_t dst = tiles_s + (uint32_t)(st * kTileBytes), fb = bar(full0 + st);
          if (leader) mbar_expect_tx(fb, (uint32_t)(nch * 2 * kChunkBytes));
          for (int ch = 0; ch < nch; ++ch) {
            // A chunk is 32 consecutive rows of the shard-major copy.  Rows past the shard's visible prefix belong
            // to later keys or, past the end of the matrix, are zero-filled: they are masked either way.
            const int slot = tab->slot0[cur.j] + cur.c * kChunk;
            if (leader) {
              tma_tile3(dst + (uint32_t)(ch * kChunkBytes), map, 0, slot, z, fb);
              tma_tile3(dst + (uint32_t)(kHalfBytes + ch * kChunkBytes), map, 64, slot, z, fb);
            }
            cur.advance(tab, n_act);
          }
          __syncwarp();
          note(8 * i + 2);
        }
      }
    }
  }
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

}  // namespace tc

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled through the runtime, so that the library does not link against the driver library.
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// Shard-major K or V copy as a 3-D tensor [batch * kv_heads][n_kv][head_dim]; box = one chunk (32 rows) x 64 columns.
bool encode_sorted(CUtensorMap* map, const void* base, int64_t n_kv, int64_t n_mats) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)tc::kD, (cuuint64_t)n_kv, (cuuint64_t)n_mats};
  const cuuint64_t strides[2] = {(cuuint64_t)tc::kD * 2, (cuuint64_t)n_kv * tc::kD * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)tc::kChunk, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Number of SMs of the current device (queried once per device).
int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

}  // namespace

cudaError_t launch_attn_tc(const AttnParams& p, const void* k_sorted, const void* v_sorted, cudaStream_t stream) {
  // the unfused route walks all KV shards of a query tile in one CTA (CASCADE_PARTIALS_WALK=0: a CTA per pair)
  const bool walk = !p.fused && CASCADE_PARTIALS_WALK && p.plan.n_kv_shards > 1;
  auto kernel = p.rope ? tc::attn_tc_kernel<true, false>
                       : (walk ? tc::attn_tc_kernel<false, true> : tc::attn_tc_kernel<false, false>);
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes);
  if (e != cudaSuccess) return e;
  tc::TmaArgs tma;
  const int64_t n_mats = (int64_t)p.batch * p.Hkv;
  if (!encode_sorted(&tma.k, k_sorted, p.plan.n_kv, n_mats) || !encode_sorted(&tma.v, v_sorted, p.plan.n_kv, n_mats)) {
    set_error("tensor-core attention: could not build the TMA descriptors of the shard-major K/V copies");
    return cudaErrorInvalidValue;
  }
  // stack as many of the G heads of a KV head into one MMA tile as divide G (at most 8)
  int lg = 0;
  while (lg < 3 && p.G % (2 << lg) == 0) ++lg;
  const int n_parts = (p.fused || walk) ? 1 : p.plan.n_kv_shards;
  const int64_t n_ctas = (int64_t)p.plan.n_qtiles[3 - lg] * (p.H >> lg) * p.batch * n_parts;
  if (n_ctas >= (int64_t)1 << 31) return cudaErrorInvalidConfiguration;
  const int tile_major = n_ctas <= 8 * (int64_t)sm_count();  // few CTAs per SM: balance matters more than L2 locality
  TimedLaunch timed(stream);
  // Programmatic dependent launch on the gather grid that precedes it in the stream: the set-up of the CTAs overlaps
  // the gather's tail.  Not while kernel timing is recording: the event between the two launches must separate them.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)n_ctas);
  cfg.blockDim = dim3(tc::kThreads);
  cfg.dynamicSmemBytes = tc::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = timing_recording() ? 0 : 1;
  e = cudaLaunchKernelEx(&cfg, kernel, p, lg, tile_major, tma);
  count_launch();
  return e;
}

}  // namespace cascade
