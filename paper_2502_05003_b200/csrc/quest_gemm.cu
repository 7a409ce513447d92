// Low-bit GEMM of the QuEST forward pass (the product step of Algorithm 1; Section 5, stage 3) for sm_100a.
//
//   acc[i][j] = sum_k cx[i][k] * cw[j][k]   exact int32, 5th-generation tensor cores
//   y[i][j]   = sx[i] * sw[j] * acc[i][j]   fused into the epilogue, bf16 or fp32 out
//
// B200 has no dense 4-bit integer MMA, so the contraction runs as tcgen05.mma kind::i8 on int8
// operand values held in a caller-provided workspace (written either by the quantizer itself or
// by unpack_codes_kernel below).  For b < 8 the operand value is 2^(7-b) times the grid value
// c = 2k-(2^b-1) (quest_operand.cuh) and the epilogue shifts the exact power of two back out;
// for b = 8 (|c| up to 255) it is v = k - 128 and the epilogue restores
// c_x . c_w = 4 v_x.v_w + 2 sum(v_x) + 2 sum(v_w) + K exactly from per-row sums.
//
// The FP4 grid (Section 4.4) has a native operand type: its packed E2M1 codes feed tcgen05.mma
// kind::mxf4 directly (MODE 5 below), with all block scales 2^0.  So do the one- and two-bit uniform
// grids, whose values +-1 and +-3 are E2M1 numbers: when both operands have at most two bits the
// workspace holds E2M1 nibbles and the same mode runs the contraction at twice the int8 rate.
//
// Two launch shapes of one kernel template.  TWO = false: one CTA per SM, persistent over 128 x BN
// output tiles.  TWO = true: clusters of two CTAs (tcgen05 cta_group::2) persistent over 256 x 256
// tiles; each CTA stages its own 128 rows of A and its own 128 of the tile's 256 rows of B, the
// leader CTA issues one M=256 MMA that reads both CTAs' shared memory, and each CTA's TMEM holds
// its 128 accumulator rows.  That cuts the operand bytes a CTA pulls from L2 per MAC by a third,
// which is what bounds the single-CTA shape.  No TMA multicast is used: every CTA loads only tiles
// it alone needs.
//
// Kernel structure:
//   warp 0      TMA producer: 128B-swizzled K-major tiles of A (128 x 128 B) and B (BN or BN/2 rows
//               x 128 B) into a 3..6-stage shared-memory ring, completion on mbarriers
//   warp 1      MMA issuer: one thread issues tcgen05.mma (M=128 or 256, N=BN, K=32) x 4 per stage
//               into one of two TMEM accumulator buffers; tcgen05.commit releases the stage /
//               signals the epilogue
//   warps 2..9  epilogue: each warp reads its 32 rows x BN/2 columns with tcgen05.ld, hands the TMEM
//               buffer back at once, then applies the integer correction and the scales, converts,
//               stages 32 x 128-byte slabs in shared memory and stores them with TMA tile stores;
//               overlaps the next tile's main loop through the second TMEM buffer
// Every wait is bounded: on expiry the CTA records a status word, stops issuing work and exits
// through the common tail (which frees its TMEM).
#include <cuda.h>
#include <cuda_bf16.h>

#include "quest_internal.cuh"
#include "quest_operand.cuh"

namespace quest {
namespace {

constexpr int BM = 128;          // tile rows (TMEM lanes)
constexpr int BK = 128;          // bytes (= int8 elements) of K per pipeline stage: one swizzle row
constexpr int UMMA_K = 32;       // K per tcgen05.mma kind::i8
constexpr int STAGES = 4;
constexpr int EPI_WARPS = 8;     // two per TMEM lane quarter, each taking half of the tile's columns
constexpr int NUM_THREADS = 64 + 32 * EPI_WARPS;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;   // ~2 s at 2 GHz

enum { ST_OK = 0, ST_PRODUCER = 1, ST_MMA = 2, ST_EPILOGUE = 3 };

struct GemmParams {
    int M, N, K;           // K: bytes of the contraction per operand row (int8: elements; bf16: 2 x elements)
    const float *sx;
    const float *sw;
    const int32_t *rs_a;   // row sums of the A operand values (nullable)
    const int32_t *rs_b;   // row sums of the B operand values (nullable)
    int mul;               // acc' = (mul*acc + ca*rs_a[i] + cb*rs_b[j] + ck) >> sh   (exact)
    int ca, cb, ck, sh;
    void *y;
    int y_dtype;
    long long ldy;
    int32_t *acc;
    const uint8_t *mask;   // backward mode: trust-mask bitmap of the output, [M x N/8] bytes (1 = keep)
    int *status;
    // SwiGLU mode: the B operand holds the gate rows [0, N) and, from row up_row0 on, the up rows; sw / rs_b
    // index the gate rows, sw2 the up rows (rs_b is one array over all rows of B)
    const float *sw2;
    int up_row0;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if the CTA is aborting or the limit expired (then it records
// `code` in the device status word and raises the CTA-wide abort flag).
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                       int *status, int code, long long limit_cycles = WAIT_LIMIT_CYCLES) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t it = 0; it < 0x7fffffffu; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 15u) == 15u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > limit_cycles) break;
        }
    }
    *abort_flag = 1;
    atomicExch(status, code);
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes,
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);          // start address, bits [0,14)
    d |= (uint64_t)1 << 16;                                // leading byte offset (unused with swizzle), bits [16,30)
    d |= (uint64_t)(1024 >> 4) << 32;                      // stride byte offset, bits [32,46)
    d |= (uint64_t)1 << 46;                                // descriptor version (sm_100), bits [46,48)
    d |= (uint64_t)2 << 61;                                // layout: SWIZZLE_128B, bits [61,64)
    return d;
}
// The same for an MN-major 16-bit operand as TMA lays it out: rows of 128 bytes hold 64 consecutive
// elements of the M (or N) dimension for one k; eight consecutive k form a 1024-byte swizzle atom;
// the next eight k follow 1024 bytes later (stride byte offset), the next 64 elements of M / N
// 8192 bytes later (leading byte offset: one 64 x 64 chunk).
__device__ __forceinline__ uint64_t make_smem_desc_mn(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
    d |= (uint64_t)(8192 >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor for kind::i8: D = s32, A = B = signed 8-bit, both K-major.
__host__ __device__ constexpr uint32_t make_idesc_i8(int m, int n) {
    return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// kind::f16 with bfloat16 operands (both K-major) and binary32 accumulation
__host__ __device__ constexpr uint32_t make_idesc_bf16(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// kind::mxf4 (Section 4.4, FP4): A and B are packed E2M1 (two per byte, K-major, 64 elements of K per
// instruction), accumulation in binary32, one UE8M0 scale per 32 elements of K read from tensor
// memory.  The low-bit path uses no block scales, so every scale byte is 2^0.
__host__ __device__ constexpr uint32_t make_idesc_mxf4(int m, int n) {
    return (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | (1u << 23) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma_mxf4(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate, uint32_t sfa_tmem, uint32_t sfb_tmem) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
        : "memory");
}
__device__ __forceinline__ void umma_mxf4_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate, uint32_t sfa_tmem, uint32_t sfb_tmem) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.block32 [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
        : "memory");
}
// Four columns of this warp's 32 tensor-memory lanes <- one word each.
__device__ __forceinline__ void tmem_st4(uint32_t taddr, uint32_t v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};" ::"r"(taddr), "r"(v), "r"(v), "r"(v), "r"(v)
                 : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The two halves of the cluster barrier on their own: a warp arrives as soon as it has nothing left to publish to
// the peer CTA and waits only where it needs the peer, so the barrier's latency overlaps the work between.
__device__ __forceinline__ void cluster_arrive() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// cta_group::2 forms: the load may signal an mbarrier of the peer CTA; the MMA spans both CTAs of
// the pair; the commit arrives on the same barrier offset in every CTA named by the mask.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *tm, int c0, int c1, uint32_t cluster_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(cluster_bar), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void umma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3)
                 : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

constexpr int MAX_STAGES = 6;

// Tile order: m fastest inside bands of RASTER_M row tiles, bands one after another.  Concurrent CTAs
// then share one or two column tiles of B while the rows of A a band touches (RASTER_M x TILE_M x K
// bytes) stay in L2 for all of the band's column tiles; with a single band (up to RASTER_M row tiles)
// this is plain column-major order.
constexpr int RASTER_M = 16;
__device__ __forceinline__ void tile_coords(int tile, int num_m, int num_n, int &tm, int &tn) {
    const int band_tiles = RASTER_M * num_n;
    const int band = tile / band_tiles;
    const int t = tile - band * band_tiles;
    const int rows_here = min(RASTER_M, num_m - band * RASTER_M);
    tn = t / rows_here;
    tm = band * RASTER_M + (t - tn * rows_here);
}

// 32 columns of this warp's 32 TMEM lanes, issued without waiting: the registers are valid only
// after tmem_wait_ld() and pin() (an empty volatile asm that makes every later use depend on a
// statement ordered after the wait).
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t *r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void pin(uint32_t &v) { asm volatile("" : "+r"(v)::"memory"); }

// Shared memory of a CTA, from a 1024-byte-aligned base: output staging, barriers, the column-scale tiles (and the
// column corrections of 8-bit codes, CBT), then the operand ring.  The ring takes as many stages as the launch's
// dynamic shared memory holds behind the alignment padding, up to MAX_NSTAGES: the kernel counts them at run time
// (a pair kernel with 256 columns gets six when the base needs no padding and no correction tile is wanted, else
// five).  A lone pair saturates with four stages; with every pair loading, the fifth is worth 4-9 % and the sixth
// another 1-2 %.
constexpr int SMEM_OPTIN_MAX = 232448;           // largest dynamic shared memory of a CTA on this part
template <int BN, bool TWO, bool CBT>
struct SmemLayout {
    static constexpr int MAX_NSTAGES = TWO ? MAX_STAGES : STAGES;     // a single CTA with 256 columns (48 KB stages) gets four when the base needs no padding, else three
    static constexpr int A_BYTES = BM * BK;
    static constexpr int B_ROWS = TWO ? BN / 2 : BN;         // rows of B this CTA stages
    static constexpr int B_BYTES = B_ROWS * BK;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int SLABS = (BN == 128) ? 2 : 1;        // what the stages leave room for
    static constexpr int STG_OFFSET = 0;                     // [8 warps][SLABS][32 rows x 128 B] output staging
    static constexpr int STG_BYTES = EPI_WARPS * SLABS * 4096;
    static constexpr int BAR_OFFSET2 = STG_OFFSET + STG_BYTES;
    static constexpr int SW_OFFSET = BAR_OFFSET2 + 256;      // [2][BN] column scales
    static constexpr int CB_OFFSET = SW_OFFSET + 2 * BN * 4; // [2][BN] column corrections (8-bit codes)
    static constexpr int RING_OFFSET = (CB_OFFSET + (CBT ? 2 * BN * 4 : 0) + 1023) / 1024 * 1024;
    static constexpr int WANTED = RING_OFFSET + MAX_NSTAGES * STAGE_BYTES + 1024;   // + slack for 1024-byte alignment
    static constexpr int TOTAL = WANTED > SMEM_OPTIN_MAX ? SMEM_OPTIN_MAX : WANTED;
    static_assert(RING_OFFSET + 2 * STAGE_BYTES + 1024 <= TOTAL, "at least two stages must fit");
};

// YT: y leaves through shared memory and TMA tile stores (whole 128-byte row segments per
// transaction) instead of per-thread 16-byte stores, which write every 32-byte sector twice.
// MODE 0: int8 operands, scaled output.  MODE 1: int8 operands with the exact correction for 8-bit
// codes.  MODE 2 (backward pass, Algorithm 2): bfloat16 operands (kind::f16, binary32 accumulators);
// the epilogue zeroes the elements the trust mask rejects and stores binary32.  MODE 3: MODE 2 plus
// the inverse Hadamard transform for blocks of 128 fused into the epilogue (BN = 256: the 128
// columns a thread holds are exactly one block), output in the caller's type.  MODE 4 (weight-only
// variant): bfloat16 operands, y = sw[n] * accumulator.  MODE 5 (FP4 grid): packed E2M1 operands on
// kind::mxf4 with unit block scales; the binary32 accumulators hold sum v_x v_w exactly (multiples of
// 1/4 below 2^22), reported as acc4 = 4 * sum; tensor memory holds one accumulator buffer of 256
// columns (or two of 128) and the scale bytes.
// OPL (bfloat16 modes only): 0 = both operands K-major; 1 = B MN-major (its memory rows run along the
// contraction); 2 = A and B MN-major.  The backward pass uses 1 and 2 to read dy and the dequantised
// operands as they lie in memory, without transposed copies.
// SWIGLU (integer modes 0, 1, 5 with BN = 256 and the TMA-store epilogue): the 256 accumulator columns
// of a tile are 128 columns of the gate projection followed by the SAME 128 columns of the up
// projection (the B operand stacks the rows of w_gate and w_up), every epilogue thread holds gate and
// up of 64 output columns of its row, and the tile leaves as h = silu(gate) * up in bfloat16: the
// MLP block's gate and up products never reach memory.
// SHORT (pair kernels of mode 0 with bfloat16 output through TMA stores and no raw accumulators): the instantiation
// for launches in which a CTA pair runs at most two tiles, where set-up and exit are a visible share.  Each warp
// arrives at the two cluster barriers as early as it can and waits as late as it can, and the output type and the
// absence of the accumulator output are constants.  With many tiles per pair the plain form measured faster.
template <int BN, int MODE, bool TWO, bool YT, int OPL = 0, bool SWIGLU = false, bool SHORT = false>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmY, GemmParams p) {
    using L = SmemLayout<BN, TWO, MODE == 1>;
    constexpr bool CORR = MODE == 1;
    constexpr bool BWD = MODE == 2 || MODE == 3;
    constexpr bool F16 = MODE >= 2;               // bfloat16 operands, binary32 accumulators
    constexpr bool WO = MODE == 4;
    constexpr bool MX = MODE == 5;
    constexpr int NBUF = (MX && BN == 256) ? 1 : 2;   // accumulator buffers in tensor memory
    constexpr uint32_t SF_COL = 256;              // MX: 32 columns of scale bytes after the accumulators
    constexpr bool IHT128 = MODE == 3;
    constexpr bool AMN = OPL == 2, BMN = OPL >= 1;
    static_assert(OPL == 0 || MODE == 2 || MODE == 3, "MN-major operands: bfloat16 backward modes only");
    static_assert(!IHT128 || BN == 256, "the fused inverse transform needs 128 columns per thread");
    static_assert(!SWIGLU || (BN == 256 && YT && (MODE == 0 || MODE == 1 || MODE == 5)), "SwiGLU epilogue: integer modes, 256 columns, TMA stores");
    static_assert(!SHORT || (TWO && MODE == 0 && YT && !SWIGLU && OPL == 0), "the short-launch form: plain int8 pair kernel");
    constexpr int BN_OUT = SWIGLU ? BN / 2 : BN;  // output columns per tile
    constexpr int TILE_M = TWO ? 2 * BM : BM;    // rows of one output tile (both CTAs of a pair)
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // 1024-byte aligned, still a shared pointer
    // stages of the operand ring that fit behind the padding (the same in every CTA of the launch: the base is a
    // property of the kernel image)
    int STAGES;
    {
        uint32_t dyn;
        asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
        const int room = (int)dyn - (int)(smem - smem_raw) - L::RING_OFFSET;
        STAGES = room / L::STAGE_BYTES;
        if (STAGES > L::MAX_NSTAGES) STAGES = L::MAX_NSTAGES;
        if (STAGES < 2) {                        // a launch with too little shared memory: refuse, touch nothing
            if (threadIdx.x == 0) atomicExch(p.status, ST_PRODUCER);
            return;
        }
    }
    uint8_t *ring = smem + L::RING_OFFSET;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::BAR_OFFSET2);
    uint64_t *full_bar = bars;                   // [STAGES] TMA -> MMA
    uint64_t *empty_bar = bars + MAX_STAGES;     // [STAGES] MMA -> TMA
    uint64_t *tfull_bar = bars + 2 * MAX_STAGES;     // [2] MMA -> epilogue
    uint64_t *tempty_bar = bars + 2 * MAX_STAGES + 2;  // [2] epilogue -> MMA
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * MAX_STAGES + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    float *sw_tile = reinterpret_cast<float *>(smem + L::SW_OFFSET);
    int32_t *cb_tile = reinterpret_cast<int32_t *>(smem + L::CB_OFFSET);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    constexpr uint32_t TMEM_COLS = MX ? 512 : 2 * BN;       // two accumulator buffers (MX: accumulators + scales)
    // pair variant: rank of this CTA in its cluster of two; rank 0 leads (issues the MMAs, owns the
    // full and accumulator-empty barriers that both CTAs signal)
    const uint32_t rank = TWO ? cluster_ctarank() : 0u;
    const bool leader = rank == 0;
    pdl_launch_dependents();
    if (threadIdx.x == 32) {
        // the TMA unit fetches a descriptor on first use: start those fetches now, while the kernel sets up
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmB)) : "memory");
        if constexpr (YT) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmY)) : "memory");
    }
    const int unit = TWO ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;          // tile-loop index
    const int num_units = TWO ? (int)(gridDim.x >> 1) : (int)gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 1);
            mbar_init(smem_u32(&empty_bar[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&tfull_bar[b]), 1);
            mbar_init(smem_u32(&tempty_bar[b]), TWO ? 2 * EPI_WARPS : EPI_WARPS);   // epilogue warps (of both CTAs of a pair)
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // barriers visible to the TMA unit
    }
    if constexpr (SHORT) {
        // only warp 0 has something to publish to the peer (the initialised barriers): every warp arrives at the
        // cluster barrier now and waits after the TMEM allocation
        __syncwarp();
        cluster_arrive();
    }
    if (warp == 1) {
        if constexpr (TWO) {      // executed by this warp of both CTAs of the pair
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                         "r"(TMEM_COLS)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                         "r"(TMEM_COLS)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (SHORT) cluster_wait();         // the peer's barriers are initialised before anything signals them
    else if constexpr (TWO) cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if constexpr (MX) {
        // unit scales: every byte of 32 columns in all 128 lanes is UE8M0 127 = 2^0 (A's scales are read
        // from the first 16 columns, B's from the second 16)
        if (warp >= 2 && warp < 6) {
            const uint32_t t_sf = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + SF_COL;
#pragma unroll
            for (int c = 0; c < 32; c += 4) tmem_st4(t_sf + (uint32_t)c, 0x7F7F7F7Fu);
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
        tc_fence_before();
        __syncthreads();
        if constexpr (TWO) cluster_sync_all();   // the leader's MMAs read the scales of both CTAs
        tc_fence_after();
    }
    pdl_wait();     // set-up above overlaps the previous kernel; operands and outputs are touched only from here

    const int num_m = (p.M + TILE_M - 1) / TILE_M;
    const int num_n = (p.N + BN_OUT - 1) / BN_OUT;
    const int num_tiles = num_m * num_n;
    const int num_kb = (p.K + BK - 1) / BK;
    // SHORT, leaving: a CTA must stay until its peer can no longer signal its barriers or read its shared and tensor
    // memory.  An epilogue warp arrives at the cluster barrier right after handing back its last accumulator buffer
    // (its last signal to the peer), the other warps after their loops, and everyone waits at the very end.
    [[maybe_unused]] bool left = false;

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = unit; tile < num_tiles && ok; tile += num_units) {
                int tm, tn;
                tile_coords(tile, num_m, num_n, tm, tn);
                const int m0 = tm * TILE_M + (int)rank * BM;                     // this CTA's rows of A
                // this CTA's rows of B (SwiGLU pair: the leader stages the gate rows, its peer the up rows)
                const int n0 = SWIGLU ? tn * BN_OUT + (int)rank * p.up_row0 : tn * BN + (int)rank * L::B_ROWS;
                for (int kb = 0; kb < num_kb; ++kb) {
                    ok = mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, abort_flag, p.status, ST_PRODUCER);
                    if (!ok) break;
                    const uint32_t fb = smem_u32(&full_bar[stage]);
                    uint8_t *sa = ring + stage * L::STAGE_BYTES;
                    // K-major: one box of 128 bytes of K x rows.  MN-major: 64 x 64 chunks (128 bytes of the
                    // M / N dimension x 64 k), 8192 bytes each, in the order of the M / N dimension.
                    if constexpr (TWO) {
                        // both CTAs' loads complete on the leader's barrier, which expects the bytes of both
                        if (leader) mbar_expect_tx(fb, 2 * L::STAGE_BYTES);
                        const uint32_t lfb = mapa_shared(fb, 0);
                        if constexpr (AMN) {
#pragma unroll
                            for (int c = 0; c < BM / 64; ++c)
                                tma_load_2d_pair(smem_u32(sa + c * 8192), &tmA, (m0 + 64 * c) * 2, kb * 64, lfb);
                        } else {
                            tma_load_2d_pair(smem_u32(sa), &tmA, kb * BK, m0, lfb);
                        }
                        if constexpr (BMN) {
#pragma unroll
                            for (int c = 0; c < L::B_ROWS / 64; ++c)
                                tma_load_2d_pair(smem_u32(sa + L::A_BYTES + c * 8192), &tmB, (n0 + 64 * c) * 2, kb * 64, lfb);
                        } else {
                            tma_load_2d_pair(smem_u32(sa + L::A_BYTES), &tmB, kb * BK, n0, lfb);
                        }
                    } else {
                        mbar_expect_tx(fb, L::STAGE_BYTES);
                        if constexpr (AMN) {
#pragma unroll
                            for (int c = 0; c < BM / 64; ++c)
                                tma_load_2d(smem_u32(sa + c * 8192), &tmA, (m0 + 64 * c) * 2, kb * 64, fb);
                        } else {
                            tma_load_2d(smem_u32(sa), &tmA, kb * BK, m0, fb);
                        }
                        if constexpr (BMN) {
#pragma unroll
                            for (int c = 0; c < L::B_ROWS / 64; ++c)
                                tma_load_2d(smem_u32(sa + L::A_BYTES + c * 8192), &tmB, (n0 + 64 * c) * 2, kb * 64, fb);
                        } else if constexpr (SWIGLU) {         // two boxes of 128 rows: gate rows, then up rows
                            tma_load_2d(smem_u32(sa + L::A_BYTES), &tmB, kb * BK, n0, fb);
                            tma_load_2d(smem_u32(sa + L::A_BYTES + (BN / 2) * BK), &tmB, kb * BK, n0 + p.up_row0, fb);
                        } else {
                            tma_load_2d(smem_u32(sa + L::A_BYTES), &tmB, kb * BK, n0, fb);
                        }
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // aborting: let copies that are still in flight land before the CTA retires
                for (int s = 0; s < STAGES; ++s) {
                    const long long t0 = clock64();
                    while (clock64() - t0 < 200000) { /* bounded drain window */ }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && leader) {
            constexpr uint32_t idesc = MX ? make_idesc_mxf4(TILE_M, BN)
                                          : F16 ? (make_idesc_bf16(TILE_M, BN) | (AMN ? 1u << 15 : 0u) | (BMN ? 1u << 16 : 0u))
                                                : make_idesc_i8(TILE_M, BN);
            int stage = 0;
            uint32_t phase = 0;
            int t = 0;
            bool ok = true;
            for (int tile = unit; tile < num_tiles && ok; tile += num_units, ++t) {
                const int buf = NBUF == 2 ? (t & 1) : 0;
                const uint32_t bphase = (uint32_t)(NBUF == 2 ? (t >> 1) : t) & 1u;
                ok = mbar_wait(smem_u32(&tempty_bar[buf]), bphase ^ 1u, abort_flag, p.status, ST_MMA);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                for (int kb = 0; kb < num_kb; ++kb) {
                    ok = mbar_wait(smem_u32(&full_bar[stage]), phase, abort_flag, p.status, ST_MMA);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sa = smem_u32(ring + stage * L::STAGE_BYTES);
                    const uint64_t a_desc = AMN ? make_smem_desc_mn(sa) : make_smem_desc(sa);
                    const uint64_t b_desc = BMN ? make_smem_desc_mn(sa + L::A_BYTES) : make_smem_desc(sa + L::A_BYTES);
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                        // advance along K: K-major +32 bytes inside the 128-byte swizzle row (+2 in 16-byte units);
                        // MN-major 16 k = two 1024-byte atoms further (+128)
                        const uint64_t ad = a_desc + (uint64_t)(kk * (AMN ? 128 : (UMMA_K >> 4)));
                        const uint64_t bd = b_desc + (uint64_t)(kk * (BMN ? 128 : (UMMA_K >> 4)));
                        const uint32_t accum = (kb | kk) != 0 ? 1u : 0u;
                        if constexpr (MX) {       // 32 bytes of K = 64 E2M1 per instruction
                            if constexpr (TWO) umma_mxf4_pair(d_tmem, ad, bd, idesc, accum, tmem_base + SF_COL, tmem_base + SF_COL + 16);
                            else umma_mxf4(d_tmem, ad, bd, idesc, accum, tmem_base + SF_COL, tmem_base + SF_COL + 16);
                        } else if constexpr (F16) {      // 32 bytes of K = 16 bfloat16 per instruction
                            if constexpr (TWO) umma_bf16_pair(d_tmem, ad, bd, idesc, accum);
                            else umma_bf16(d_tmem, ad, bd, idesc, accum);
                        } else {
                            if constexpr (TWO) umma_i8_pair(d_tmem, ad, bd, idesc, accum);
                            else umma_i8(d_tmem, ad, bd, idesc, accum);
                        }
                    }
                    // stage reusable (in both CTAs of a pair) once these MMAs retire
                    if constexpr (TWO) umma_commit_pair(smem_u32(&empty_bar[stage]));
                    else umma_commit(smem_u32(&empty_bar[stage]));
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) {                                          // accumulator complete
                    if constexpr (TWO) umma_commit_pair(smem_u32(&tfull_bar[buf]));
                    else umma_commit(smem_u32(&tfull_bar[buf]));
                }
            }
        }
        __syncwarp();
    } else {
        // ---- epilogue: 8 warps; warp w reads TMEM lanes [32 (w & 3), +32) = tile rows 32 (w & 3) + lane
        //      and the column half (w - 2) / 4 of the tile ------------------------------------------------
        constexpr int CW = BN / 2;                     // columns per warp
        const int quarter = warp & 3;
        const int hgrp = (warp - 2) >> 2;              // which half of the tile's (output) columns
        const int cbase = hgrp * CW;
        // plain modes: a warp takes CW consecutive accumulator columns; SwiGLU: gate columns [64 hgrp, +64) and
        // the up columns of the same outputs, 128 further on
        const int ep_tid = threadIdx.x - 64;           // 0..255 over the epilogue warps
        int t = 0;
        bool ok = true;
        const bool vec_y = p.y && (((reinterpret_cast<uintptr_t>(p.y) & 15) == 0) &&
                                   (p.ldy % (p.y_dtype == QUEST_BF16 ? 8 : 4) == 0));
        const bool vec_acc = !SHORT && p.acc && (p.N % 4 == 0) && ((reinterpret_cast<uintptr_t>(p.acc) & 15) == 0);
        const bool y_f32 = !SHORT && p.y_dtype == QUEST_F32;
        uint8_t *slab_base = smem + L::STG_OFFSET + (warp - 2) * (L::SLABS * 4096);
        int slab_count = 0;                            // slabs this warp has handed to TMA
        for (int tile = unit; tile < num_tiles && ok; tile += num_units, ++t) {
            int tm, tn;
            tile_coords(tile, num_m, num_n, tm, tn);
            const int m0 = tm * TILE_M + (int)rank * BM;
            const int n0 = tn * BN_OUT;
            const int buf = NBUF == 2 ? (t & 1) : 0;
            const uint32_t bphase = (uint32_t)(NBUF == 2 ? (t >> 1) : t) & 1u;
            // stage this tile's column scales (and column corrections) in shared memory; the
            // buffer of tile t was last read during tile t-2, which every warp left before it
            // arrived at the barrier of tile t-1
            float *swt = sw_tile + (t & 1) * BN;
            int32_t *cbt = cb_tile + (t & 1) * BN;
            for (int c = ep_tid; c < BN; c += 32 * EPI_WARPS) {
                if constexpr (SWIGLU) {
                    const bool up = c >= BN_OUT;
                    const int col = n0 + (up ? c - BN_OUT : c);
                    swt[c] = col < p.N ? __ldg((up ? p.sw2 : p.sw) + col) : 0.0f;
                    if (CORR) cbt[c] = (p.rs_b && col < p.N) ? p.cb * __ldg(p.rs_b + col + (up ? p.up_row0 : 0)) : 0;
                } else {
                    const int col = n0 + c;
                    if (!BWD) swt[c] = (p.y && col < p.N) ? __ldg(p.sw + col) : 0.0f;
                    if (CORR) cbt[c] = (p.rs_b && col < p.N) ? p.cb * __ldg(p.rs_b + col) : 0;
                }
            }
            const int row = m0 + quarter * 32 + lane;
            const bool row_ok = row < p.M;
            // without 8-bit corrections and without the raw accumulators, the exact power of two of the
            // operand scaling is folded into the row scale instead of shifting every accumulator
            const bool fold = SHORT || (!CORR && !p.acc);
            float sxr = WO ? 1.0f : (!BWD && row_ok && p.y) ? __ldg(p.sx + row) : 0.0f;
            if (fold) sxr = __fmul_rn(sxr, __uint_as_float((uint32_t)(127 - p.sh) << 23));
            int rsa = 0;
            if (CORR) rsa = (row_ok && p.rs_a) ? p.ca * __ldg(p.rs_a + row) + p.ck : p.ck;
            ok = mbar_wait(smem_u32(&tfull_bar[buf]), bphase, abort_flag, p.status, ST_EPILOGUE);
            // one barrier over the epilogue threads publishes the staged scales and makes the
            // continue/abort decision unanimous, so no warp can be left waiting at a later barrier
            {
                uint32_t all_ok;
                asm volatile(
                    "{\n\t.reg .pred p, q;\n\t"
                    "setp.ne.u32 q, %1, 0;\n\t"
                    "bar.red.and.pred p, 1, %2, q;\n\t"
                    "selp.u32 %0, 1, 0, p;\n\t}"
                    : "=r"(all_ok)
                    : "r"((uint32_t)(ok ? 1u : 0u)), "n"(32 * EPI_WARPS)
                    : "memory");
                ok = all_ok != 0;
            }
            if (!ok) break;
            tc_fence_after();
            // all of this warp's accumulator columns in one go, then hand the TMEM buffer back to
            // the MMA warp before any arithmetic
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN);
            uint32_t r[SWIGLU ? 1 : CW];
            auto release_tmem = [&]() {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if constexpr (TWO) mbar_arrive_cluster(mapa_shared(smem_u32(&tempty_bar[buf]), 0));   // the leader's barrier
                    else mbar_arrive(smem_u32(&tempty_bar[buf]));
                }
                if constexpr (SHORT) {
                    if (tile + num_units >= num_tiles) {       // this CTA's last tile: nothing more goes to the peer
                        __syncwarp();
                        cluster_arrive();
                        left = true;
                    }
                }
            };
            if constexpr (!SWIGLU) {
#pragma unroll
                for (int c0 = 0; c0 < CW; c0 += 32)
                    if (n0 + cbase + c0 < p.N) tmem_ld32_issue(t_row + (uint32_t)(cbase + c0), &r[c0]);     // uniform predicate
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < CW; ++j) pin(r[j]);
                release_tmem();
            }
            if constexpr (IHT128) {
                // trust mask and inverse transform of Algorithm 2 on this thread's block of 128: mask, then the inverse
                // orthonormal Hadamard transform in registers (descending stride, packed binary32)
                if (n0 + cbase < p.N) {
                    uint4 mb = make_uint4(0u, 0u, 0u, 0u);
                    if (row_ok) mb = __ldg(reinterpret_cast<const uint4 *>(p.mask + (long long)row * (p.N >> 3) + ((n0 + cbase) >> 3)));
                    const uint32_t mw4[4] = {mb.x, mb.y, mb.z, mb.w};
#pragma unroll
                    for (int j = 0; j < 128; ++j) r[j] = ((mw4[j >> 5] >> (j & 31)) & 1u) ? r[j] : 0u;
                    const float2 neg1 = make_float2(-1.0f, -1.0f);
#pragma unroll
                    for (int s2 = 32; s2 >= 1; s2 >>= 1) {          // strides 64 .. 2 in pairs of columns
#pragma unroll
                        for (int i = 0; i < 64; ++i)
                            if ((i & s2) == 0) {
                                const float2 a = make_float2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
                                const float2 b = make_float2(__uint_as_float(r[2 * (i + s2)]), __uint_as_float(r[2 * (i + s2) + 1]));
                                const float2 su = __fadd2_rn(a, b), di = __ffma2_rn(b, neg1, a);
                                r[2 * i] = __float_as_uint(su.x); r[2 * i + 1] = __float_as_uint(su.y);
                                r[2 * (i + s2)] = __float_as_uint(di.x); r[2 * (i + s2) + 1] = __float_as_uint(di.y);
                            }
                    }
                    const float2 sc = make_float2(0.08838834764831845f, 0.08838834764831845f);    // 1 / sqrt(128)
#pragma unroll
                    for (int i = 0; i < 64; ++i) {                  // stride 1, then the normalisation
                        const float a = __uint_as_float(r[2 * i]), b = __uint_as_float(r[2 * i + 1]);
                        const float2 o = __fmul2_rn(make_float2(a + b, a - b), sc);
                        r[2 * i] = __float_as_uint(o.x);
                        r[2 * i + 1] = __float_as_uint(o.y);
                    }
                }
            }
            if constexpr (SWIGLU) {
                // 64 output columns per thread, in two rounds of 32: gate and up accumulators of the round come out of
                // tensor memory together (64 registers), the buffer goes back to the MMA warp after the second load
                const int out0 = n0 + 64 * hgrp;               // first of this thread's 64 output columns
                const bool live = out0 < p.N;                  // uniform across the warp
                uint8_t *slab = slab_base;
                if (live) {
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the slab's last store has read it
                    __syncwarp();
                }
                const float2 sx2 = make_float2(sxr, sxr);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t g[32], u[32];
                    const int gc = 64 * hgrp + 32 * half, uc = 128 + gc;         // accumulator columns: gate, up
                    const bool part = out0 + 32 * half < p.N;
                    if (part) {
                        tmem_ld32_issue(t_row + (uint32_t)gc, g);
                        tmem_ld32_issue(t_row + (uint32_t)uc, u);
                    }
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) { pin(g[j]); pin(u[j]); }
                    if (half == 1) release_tmem();
                    if (part) {
                        if (CORR) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                g[j] = (uint32_t)((int32_t)((uint32_t)p.mul * g[j] + (uint32_t)rsa + (uint32_t)cbt[gc + j]) >> p.sh);
                                u[j] = (uint32_t)((int32_t)((uint32_t)p.mul * u[j] + (uint32_t)rsa + (uint32_t)cbt[uc + j]) >> p.sh);
                            }
                        }
                        const float2 *swg = reinterpret_cast<const float2 *>(swt + gc), *swu = reinterpret_cast<const float2 *>(swt + uc);
                        uint32_t packed[16];
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            const float2 ag = MX ? make_float2(__uint_as_float(g[j]), __uint_as_float(g[j + 1]))
                                                 : make_float2((float)(int32_t)g[j], (float)(int32_t)g[j + 1]);
                            const float2 au = MX ? make_float2(__uint_as_float(u[j]), __uint_as_float(u[j + 1]))
                                                 : make_float2((float)(int32_t)u[j], (float)(int32_t)u[j + 1]);
                            const float2 gv = __fmul2_rn(__fmul2_rn(sx2, swg[j >> 1]), ag);
                            const float2 uv = __fmul2_rn(__fmul2_rn(sx2, swu[j >> 1]), au);
                            // h = silu(gate) * up, silu(z) = z / (1 + exp(-z)).  The exponential and the reciprocal are the
                            // hardware approximations (a few units of 2^-23 each, no branches): exp(-z) overflows to +inf
                            // for z < -88, where the quotient is -0 as it should be.
                            float e0, e1, r0, r1;
                            asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(gv.x * -1.4426950408889634f));
                            asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(gv.y * -1.4426950408889634f));
                            asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r0) : "f"(1.0f + e0));
                            asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r1) : "f"(1.0f + e1));
                            const __nv_bfloat162 hh = __floats2bfloat162_rn((gv.x * r0) * uv.x, (gv.y * r1) * uv.y);
                            packed[j >> 1] = *reinterpret_cast<const uint32_t *>(&hh);
                        }
                        uint8_t *rowp = slab + lane * 128;
                        const int sw7 = lane & 7;
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            *reinterpret_cast<uint4 *>(rowp + (((half * 4 + j) ^ sw7) << 4)) =
                                make_uint4(packed[4 * j], packed[4 * j + 1], packed[4 * j + 2], packed[4 * j + 3]);
                    }
                }
                if (live) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        asm volatile(
                            "cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                            ::"l"(reinterpret_cast<uint64_t>(&tmY)), "r"(smem_u32(slab)), "r"(out0 * 2), "r"(m0 + quarter * 32)
                            : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                }
            }
#pragma unroll
            for (int c0 = 0; c0 < (SWIGLU ? 0 : CW); c0 += 32) {
                const int col0 = n0 + cbase + c0;
                if (col0 < p.N) {                      // uniform across the warp
                    const bool full = col0 + 32 <= p.N;
                    uint32_t *rc = &r[c0];
                    if constexpr (IHT128) {
                        // already masked and transformed above
                    } else if constexpr (BWD) {
                        // trust estimator: keep the gradient only where the forward mask trusts the element
                        const uint32_t mbits = row_ok ? __ldg(reinterpret_cast<const uint32_t *>(
                                                            p.mask + (long long)row * (p.N >> 3) + (col0 >> 3)))
                                                      : 0u;
#pragma unroll
                        for (int j = 0; j < 32; ++j) rc[j] = ((mbits >> j) & 1u) ? rc[j] : 0u;
                    } else if (CORR) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            rc[j] = (uint32_t)((int32_t)((uint32_t)p.mul * rc[j] + (uint32_t)rsa +
                                                         (uint32_t)cbt[cbase + c0 + j]) >> p.sh);
                    } else if (!MX && !fold) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) rc[j] = (uint32_t)((int32_t)rc[j] >> p.sh);
                    }
                    if (MX && p.acc && row_ok) {
                        // the accumulator is exact: an integer (uniform grids) or a multiple of 1/4 (FP4 grid, mul = 4)
                        int32_t *dst = p.acc + (long long)row * p.N + col0;
                        const float am = (float)p.mul;
                        if (vec_acc && full) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                *reinterpret_cast<int4 *>(dst + j) =
                                    make_int4(__float2int_rn(__uint_as_float(rc[j]) * am), __float2int_rn(__uint_as_float(rc[j + 1]) * am),
                                              __float2int_rn(__uint_as_float(rc[j + 2]) * am), __float2int_rn(__uint_as_float(rc[j + 3]) * am));
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (col0 + j < p.N) dst[j] = __float2int_rn(__uint_as_float(rc[j]) * am);
                        }
                    }
                    if (!SHORT && !MX && !BWD && p.acc && row_ok) {
                        int32_t *dst = p.acc + (long long)row * p.N + col0;
                        if (vec_acc && full) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                *reinterpret_cast<uint4 *>(dst + j) = make_uint4(rc[j], rc[j + 1], rc[j + 2], rc[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (col0 + j < p.N) dst[j] = (int32_t)rc[j];
                        }
                    }
                    if (p.y) {
                        // y = (sx * sw) * acc, each product rounded to binary32 (two columns per instruction)
                        const float2 sx2 = make_float2(sxr, sxr);
                        const float2 *sw2 = reinterpret_cast<const float2 *>(swt + cbase + c0);
#pragma unroll
                        for (int j = 0; j < (BWD ? 0 : 32); j += 2) {
                            const float2 a2 = (WO || MX) ? make_float2(__uint_as_float(rc[j]), __uint_as_float(rc[j + 1]))
                                                 : make_float2((float)(int32_t)rc[j], (float)(int32_t)rc[j + 1]);
                            const float2 y2 = __fmul2_rn(__fmul2_rn(sx2, sw2[j >> 1]), a2);
                            rc[j] = __float_as_uint(y2.x);
                            rc[j + 1] = __float_as_uint(y2.y);
                        }
                        if constexpr (YT) {
                            // stage 32 rows x 128 bytes (128-byte swizzle: 16-byte chunk j of row r sits at
                            // j ^ (r & 7)), then one lane stores the slab with a TMA tile store, which clips
                            // at the matrix edges.  Binary32 fills a slab per 32 columns, bfloat16 per 64.
                            const int half = y_f32 ? 0 : ((c0 >> 5) & 1);
                            uint8_t *slab = slab_base + (L::SLABS == 2 ? (slab_count & 1) * 4096 : 0);
                            if (half == 0) {
                                // the store that last used this slab must have finished reading it
                                if (lane == 0) {
                                    if (L::SLABS == 2) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                                    else asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                                }
                                __syncwarp();
                            }
                            uint8_t *rowp = slab + lane * 128;
                            const int sw7 = lane & 7;
                            if (y_f32) {
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    *reinterpret_cast<uint4 *>(rowp + ((j ^ sw7) << 4)) =
                                        make_uint4(rc[4 * j], rc[4 * j + 1], rc[4 * j + 2], rc[4 * j + 3]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    uint4 q;
                                    __nv_bfloat162 h;
                                    h = __floats2bfloat162_rn(__uint_as_float(rc[8 * j]), __uint_as_float(rc[8 * j + 1]));
                                    q.x = *reinterpret_cast<uint32_t *>(&h);
                                    h = __floats2bfloat162_rn(__uint_as_float(rc[8 * j + 2]), __uint_as_float(rc[8 * j + 3]));
                                    q.y = *reinterpret_cast<uint32_t *>(&h);
                                    h = __floats2bfloat162_rn(__uint_as_float(rc[8 * j + 4]), __uint_as_float(rc[8 * j + 5]));
                                    q.z = *reinterpret_cast<uint32_t *>(&h);
                                    h = __floats2bfloat162_rn(__uint_as_float(rc[8 * j + 6]), __uint_as_float(rc[8 * j + 7]));
                                    q.w = *reinterpret_cast<uint32_t *>(&h);
                                    *reinterpret_cast<uint4 *>(rowp + (((half * 4 + j) ^ sw7) << 4)) = q;
                                }
                            }
                            const bool flush = y_f32 || half == 1 || (col0 + 32 >= p.N);
                            if (flush) {
                                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                                __syncwarp();
                                if (lane == 0) {
                                    const int first_col = y_f32 ? col0 : col0 - half * 32;
                                    const int xbytes = first_col * (y_f32 ? 4 : 2);       // a multiple of 64
                                    asm volatile(
                                        "cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                                        ::"l"(reinterpret_cast<uint64_t>(&tmY)), "r"(smem_u32(slab)), "r"(xbytes),
                                          "r"(m0 + quarter * 32)
                                        : "memory");
                                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                                }
                                ++slab_count;
                            }
                        } else if (row_ok) {
                            if (p.y_dtype == QUEST_BF16) {
                                __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(p.y) + (long long)row * p.ldy + col0;
                                if (vec_y && full) {
#pragma unroll
                                    for (int j = 0; j < 32; j += 8) {
                                        uint4 q;
                                        __nv_bfloat162 h;
                                        h = __floats2bfloat162_rn(__uint_as_float(rc[j]), __uint_as_float(rc[j + 1]));
                                        q.x = *reinterpret_cast<uint32_t *>(&h);
                                        h = __floats2bfloat162_rn(__uint_as_float(rc[j + 2]), __uint_as_float(rc[j + 3]));
                                        q.y = *reinterpret_cast<uint32_t *>(&h);
                                        h = __floats2bfloat162_rn(__uint_as_float(rc[j + 4]), __uint_as_float(rc[j + 5]));
                                        q.z = *reinterpret_cast<uint32_t *>(&h);
                                        h = __floats2bfloat162_rn(__uint_as_float(rc[j + 6]), __uint_as_float(rc[j + 7]));
                                        q.w = *reinterpret_cast<uint32_t *>(&h);
                                        *reinterpret_cast<uint4 *>(dst + j) = q;
                                    }
                                } else {
#pragma unroll
                                    for (int j = 0; j < 32; ++j)
                                        if (col0 + j < p.N) dst[j] = __float2bfloat16_rn(__uint_as_float(rc[j]));
                                }
                            } else {
                                float *dst = reinterpret_cast<float *>(p.y) + (long long)row * p.ldy + col0;
                                if (vec_y && full) {
#pragma unroll
                                    for (int j = 0; j < 32; j += 4)
                                        *reinterpret_cast<uint4 *>(dst + j) = make_uint4(rc[j], rc[j + 1], rc[j + 2], rc[j + 3]);
                                } else {
#pragma unroll
                                    for (int j = 0; j < 32; ++j)
                                        if (col0 + j < p.N) dst[j] = __uint_as_float(rc[j]);
                                }
                            }
                        }
                    }
                }
            }
        }
    }

    if constexpr (YT) {
        // output tiles still on their way out of shared memory: the CTA may retire once the copy engine has read
        // them (the writes themselves are ordered before the end of the grid)
        if (warp >= 2 && lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    }
    tc_fence_before();
    if constexpr (SHORT) {
        __syncwarp();
        if (!left) cluster_arrive();             // uniform per warp
        cluster_wait();
    } else {
        __syncthreads();
        // a CTA of a pair must stay until its peer can no longer signal its barriers or read its
        // shared memory and tensor memory
        if constexpr (TWO) cluster_sync_all();
    }
    if (warp == 1) {
        tc_fence_after();
        if constexpr (TWO)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// Packed codes -> int8 operand values (quest_operand.cuh).  One thread converts 32 consecutive
// elements (rows are dense and K % 32 == 0).
// ---------------------------------------------------------------------------------------------
template <int CB>
__global__ void unpack_codes_kernel(const uint8_t *__restrict__ codes, int bits, long long n_groups,
                                    int8_t *__restrict__ out) {
    pdl_launch_dependents();
    pdl_wait();
    for (long long g = blockIdx.x * (long long)blockDim.x + threadIdx.x; g < n_groups;
         g += (long long)gridDim.x * blockDim.x) {
        const uint32_t *src = reinterpret_cast<const uint32_t *>(codes) + g * CB;
        uint32_t w[CB];
#pragma unroll
        for (int i = 0; i < CB; ++i) w[i] = __ldg(src + i);
        uint32_t o[8];
        operand_from_code_words<CB>(w, bits, o);
        uint4 *dst = reinterpret_cast<uint4 *>(out + g * 32);
        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

// Packed one- or two-bit codes -> E2M1 nibble operands (quest_operand.cuh), 32 elements per thread.
template <int CB>
__global__ void unpack_codes_e2m1_kernel(const uint8_t *__restrict__ codes, long long n_groups, uint8_t *__restrict__ out) {
    pdl_launch_dependents();
    pdl_wait();
    for (long long g = blockIdx.x * (long long)blockDim.x + threadIdx.x; g < n_groups;
         g += (long long)gridDim.x * blockDim.x) {
        uint32_t w[CB];
#pragma unroll
        for (int q = 0; q < CB; ++q) w[q] = __ldg(reinterpret_cast<const uint32_t *>(codes) + g * CB + q);
        uint32_t o[4];
        e2m1_operand_from_code_words<CB>(w, o);
        *reinterpret_cast<uint4 *>(out + g * 16) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// Both operands of a contraction in one launch (each with its own width): thread g converts 32
// consecutive elements of x when g < groups_x, else of w.
template <int CB>
__device__ __forceinline__ void unpack_group(const uint8_t *codes, int bits, long long g, uint8_t *out, bool e2m1) {
    uint32_t w[CB];
#pragma unroll
    for (int q = 0; q < CB; ++q) w[q] = __ldg(reinterpret_cast<const uint32_t *>(codes) + g * CB + q);
    if constexpr (CB <= 2) {
        if (e2m1) {
            uint32_t o[4];
            e2m1_operand_from_code_words<CB>(w, o);
            *reinterpret_cast<uint4 *>(out + g * 16) = make_uint4(o[0], o[1], o[2], o[3]);
            return;
        }
    }
    uint32_t o[8];
    operand_from_code_words<CB>(w, bits, o);
    uint4 *dst = reinterpret_cast<uint4 *>(out + g * 32);
    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
}
__global__ void __launch_bounds__(128)
unpack_pair_kernel(const uint8_t *__restrict__ codes_x, int bits_x, long long groups_x, uint8_t *__restrict__ out_x,
                   const uint8_t *__restrict__ codes_w, int bits_w, long long groups_w, uint8_t *__restrict__ out_w, int e2m1) {
    pdl_launch_dependents();
    pdl_wait();
    long long g = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (g >= groups_x + groups_w) return;
    const bool second = g >= groups_x;
    if (second) g -= groups_x;
    const uint8_t *codes = second ? codes_w : codes_x;
    uint8_t *out = second ? out_w : out_x;
    const int bits = second ? bits_w : bits_x;
    switch (bits == 1 ? 1 : bits == 2 ? 2 : bits <= 4 ? 4 : 8) {
        case 1: unpack_group<1>(codes, bits, g, out, e2m1 != 0); break;
        case 2: unpack_group<2>(codes, bits, g, out, e2m1 != 0); break;
        case 4: unpack_group<4>(codes, bits, g, out, false); break;
        default: unpack_group<8>(codes, bits, g, out, false); break;
    }
}

// Row sums of an int8 matrix [rows x K]: one warp per row.
__global__ void rowsum_i8_kernel(const int8_t *__restrict__ a, long long rows, int K, int32_t *__restrict__ out) {
    pdl_launch_dependents();
    pdl_wait();
    const long long row = blockIdx.x * (long long)(blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int lane = threadIdx.x & 31;
    const int8_t *r = a + row * (long long)K;
    int s = 0;
    for (int k = lane * 4; k < K; k += 128) {
        const uint32_t w = *reinterpret_cast<const uint32_t *>(r + k);
        s += (int8_t)(w & 0xff) + (int8_t)((w >> 8) & 0xff) + (int8_t)((w >> 16) & 0xff) + (int8_t)(w >> 24);
    }
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) out[row] = s;
}

// Self-test of the bounded wait: one warp waits, with a short limit, on a barrier that nothing will ever
// complete.  The wait must give up, record its code in the status word, raise the abort flag, and a second
// wait must then return at once because the CTA is aborting: the path every kernel of the library takes
// when a copy or a partner CTA fails to arrive, exercised here without any fault.
__global__ void bounded_wait_probe_kernel(long long limit_cycles, int *status, int *report) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const long long t0 = clock64();
        const bool first = mbar_wait(smem_u32(&bar), 0, &abort_flag, status, ST_PRODUCER, limit_cycles);
        const long long t1 = clock64();
        const bool second = mbar_wait(smem_u32(&bar), 0, &abort_flag, status, ST_MMA, limit_cycles);
        const long long t2 = clock64();
        if (report) {
            report[0] = first ? 1 : 0;                       // 0: the wait gave up
            report[1] = second ? 1 : 0;                      // 0: refused at once, the CTA is aborting
            report[2] = abort_flag;
            report[3] = (t2 - t1) < (t1 - t0) ? 1 : 0;       // the second wait did not run its limit out again
        }
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// Encoding a tensor map is a driver call of a microsecond or two, and a layer that is called again and again
// passes the same pointers and shapes every time.  Each host thread keeps the last few descriptors it built, keyed
// by everything that goes into them (a descriptor is a pure function of its key, so a hit is always valid).
struct MapKey {
    const void *base;
    int64_t d0, d1, pitch;
    int box0, box1, swizzle, promo;
    bool operator==(const MapKey &o) const {
        return base == o.base && d0 == o.d0 && d1 == o.d1 && pitch == o.pitch && box0 == o.box0 && box1 == o.box1 &&
               swizzle == o.swizzle && promo == o.promo;
    }
};
struct MapCache {
    static constexpr int N = 16;
    MapKey key[N];
    CUtensorMap map[N];
    int used = 0, next = 0;
    const CUtensorMap *find(const MapKey &k) const {
        for (int i = 0; i < used; ++i)
            if (key[i] == k) return &map[i];
        return nullptr;
    }
    void put(const MapKey &k, const CUtensorMap &m) {
        key[next] = k;
        map[next] = m;
        next = (next + 1) % N;
        if (used < N) ++used;
    }
};
static thread_local MapCache t_map_cache;

// int8 matrix [rows x K], K contiguous; box = 128 bytes of K x box_rows rows, 128-byte swizzle.
int make_operand_map(CUtensorMap *tm, const int8_t *base, int64_t rows, int64_t K, int box_rows) {
    const MapKey mk = {base, K, rows, K, BK, box_rows, 1, 1};
    if (const CUtensorMap *hit = t_map_cache.find(mk)) { *tm = *hit; return QUEST_OK; }
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return cuda_fail_msg("cuTensorMapEncodeTiled entry point not available");
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cuda_fail_msg("cuTensorMapEncodeTiled failed");
    t_map_cache.put(mk, *tm);
    return QUEST_OK;
}

// y viewed as bytes: [rows x row_bytes], row pitch pitch_bytes; box = 128 bytes x 32 rows, 128-byte swizzle.
int make_output_map(CUtensorMap *tm, void *base, int64_t rows, int64_t row_bytes, int64_t pitch_bytes) {
    const MapKey mk = {base, row_bytes, rows, pitch_bytes, 128, 32, 1, 0};
    if (const CUtensorMap *hit = t_map_cache.find(mk)) { *tm = *hit; return QUEST_OK; }
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return cuda_fail_msg("cuTensorMapEncodeTiled entry point not available");
    cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)pitch_bytes};
    cuuint32_t box[2] = {128, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cuda_fail_msg("cuTensorMapEncodeTiled failed for the output");
    t_map_cache.put(mk, *tm);
    return QUEST_OK;
}

template <int BN, int MODE, bool TWO, bool YT, int OPL = 0, bool SWIGLU = false, bool SHORT = false>
int launch_gemm_bn(const CUtensorMap &tmA, const CUtensorMap &tmB, const CUtensorMap &tmY, const GemmParams &p,
                   cudaStream_t st) {
    using L = SmemLayout<BN, TWO, MODE == 1>;
    static DynamicSmemOnce smem_attr;            // per kernel instantiation, per device
    {
        cudaError_t e = smem_attr.set(gemm_i8_kernel<BN, MODE, TWO, YT, OPL, SWIGLU, SHORT>, L::TOTAL);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int tile_m = TWO ? 2 * BM : BM;
    const int bn_out = SWIGLU ? BN / 2 : BN;
    const int tiles = ((p.M + tile_m - 1) / tile_m) * ((p.N + bn_out - 1) / bn_out);
    int grid;
    if (TWO) {
        const int pairs = tiles < sms / 2 ? tiles : sms / 2;
        grid = 2 * pairs;
    } else {
        grid = tiles < sms ? tiles : sms;
    }
    cudaError_t e = launch_pdl(gemm_i8_kernel<BN, MODE, TWO, YT, OPL, SWIGLU, SHORT>, dim3((unsigned)grid), dim3(NUM_THREADS), (size_t)L::TOTAL, st,
                               TWO ? 2 : 1, tmA, tmB, tmY, p);
    return e == cudaSuccess ? QUEST_OK : cuda_fail(e);
}

}  // namespace

int launch_bounded_wait_probe(long long limit_cycles, int *report, cudaStream_t st) {
    int *status = device_status_word();
    if (!status) return QUEST_ERR_CUDA;
    bounded_wait_probe_kernel<<<1, 32, 0, st>>>(limit_cycles, status, report);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? QUEST_OK : cuda_fail(e);
}

// The operand of w and its row sums come first, so that their place does not depend on M: a caller
// that keeps the workspace can reuse w's operand across calls with different numbers of rows of x.
Workspace carve_workspace(void *base, int64_t M, int64_t N, int64_t K) {
    Workspace w;
    size_t off = 0;
    uint8_t *b = reinterpret_cast<uint8_t *>(base);
    w.b8 = reinterpret_cast<int8_t *>(b + off);
    off += align_up((size_t)(N * K), 256);
    w.rs_b = reinterpret_cast<int32_t *>(b + off);
    off += align_up((size_t)N * 4, 256);
    w.a8 = reinterpret_cast<int8_t *>(b + off);
    off += align_up((size_t)(M * K), 256);
    w.rs_a = reinterpret_cast<int32_t *>(b + off);
    off += align_up((size_t)M * 4, 256);
    w.bytes = off;
    return w;
}

int launch_unpack(const uint8_t *codes, int bits, int64_t rows, int64_t K, int8_t *out, int32_t *rowsum,
                  cudaStream_t st, bool e2m1) {
    if (rows == 0) return QUEST_OK;
    const long long n_groups = rows * K / 32;
    const int threads = 256;
    long long blocks = (n_groups + threads - 1) / threads;
    if (blocks > 148 * 16) blocks = 148 * 16;
    cudaError_t e;
    if (e2m1) {                                       // bits <= 2: nibble operands, [rows x K/2] bytes
        uint8_t *o4 = reinterpret_cast<uint8_t *>(out);
        if (bits == 1) e = launch_pdl(unpack_codes_e2m1_kernel<1>, dim3((unsigned)blocks), dim3(threads), 0, st, 1, codes, n_groups, o4);
        else e = launch_pdl(unpack_codes_e2m1_kernel<2>, dim3((unsigned)blocks), dim3(threads), 0, st, 1, codes, n_groups, o4);
        return e == cudaSuccess ? QUEST_OK : cuda_fail(e);
    }
    switch (container_bits(bits)) {
        case 1: e = launch_pdl(unpack_codes_kernel<1>, dim3((unsigned)blocks), dim3(threads), 0, st, 1, codes, bits, n_groups, out); break;
        case 2: e = launch_pdl(unpack_codes_kernel<2>, dim3((unsigned)blocks), dim3(threads), 0, st, 1, codes, bits, n_groups, out); break;
        case 4: e = launch_pdl(unpack_codes_kernel<4>, dim3((unsigned)blocks), dim3(threads), 0, st, 1, codes, bits, n_groups, out); break;
        default: e = launch_pdl(unpack_codes_kernel<8>, dim3((unsigned)blocks), dim3(threads), 0, st, 1, codes, bits, n_groups, out); break;
    }
    if (e != cudaSuccess) return cuda_fail(e);
    if (rowsum) return launch_rowsum(out, rows, K, rowsum, st);
    return QUEST_OK;
}

int launch_unpack_pair(const uint8_t *xq, int bits_x, int64_t M, int8_t *a8, int32_t *rs_a,
                       const uint8_t *wq, int bits_w, int64_t N, int8_t *b8, int32_t *rs_b, int64_t K, bool e2m1,
                       cudaStream_t st) {
    const long long gx = M * K / 32, gw = N * K / 32;
    if (gx + gw == 0) return QUEST_OK;
    cudaError_t e = launch_pdl(unpack_pair_kernel, dim3((unsigned)((gx + gw + 127) / 128)), dim3(128), 0, st, 1, xq, bits_x, gx,
                               reinterpret_cast<uint8_t *>(a8), wq, bits_w, gw, reinterpret_cast<uint8_t *>(b8), e2m1 ? 1 : 0);
    if (e != cudaSuccess) return cuda_fail(e);
    int s = QUEST_OK;
    if (rs_a) s = launch_rowsum(a8, M, K, rs_a, st);
    if (!s && rs_b) s = launch_rowsum(b8, N, K, rs_b, st);
    return s;
}

int launch_rowsum(const int8_t *a8, int64_t rows, int64_t K, int32_t *rowsum, cudaStream_t st) {
    if (rows == 0) return QUEST_OK;
    const long long rb = (rows + 7) / 8;
    cudaError_t e = launch_pdl(rowsum_i8_kernel, dim3((unsigned)rb), dim3(256), 0, st, 1, a8, (long long)rows, (int)K, rowsum);
    return e == cudaSuccess ? QUEST_OK : cuda_fail(e);
}

int launch_gemm(const int8_t *a8, const int8_t *b8, const int32_t *rs_a, const int32_t *rs_b,
                int bits_x, int bits_w, const float *sx, const float *sw,
                int64_t M, int64_t N, int64_t K, void *y, int y_dtype, int64_t ldy,
                int32_t *acc, cudaStream_t st) {
    if (M == 0 || N == 0) return QUEST_OK;
    if (e2m1_operands(bits_x, bits_w))               // both operands are E2M1 nibbles of the grid values
        return launch_gemm_e2m1(reinterpret_cast<const uint8_t *>(a8), reinterpret_cast<const uint8_t *>(b8), sx, sw, M, N, K,
                                y, y_dtype, ldy, acc, 1, st);
    // operand value v relates to the grid value c by v = 2^(7-b) c below 8 bits and c = 2v + 1 at 8 bits
    const bool x8 = bits_x == 8, w8 = bits_w == 8;
    GemmParams p;
    p.M = (int)M; p.N = (int)N; p.K = (int)K;
    p.sx = sx; p.sw = sw;
    if (!x8 && !w8) { p.mul = 1; p.ca = 0; p.cb = 0; p.ck = 0; p.sh = 14 - bits_x - bits_w; }
    else if (x8 && w8) { p.mul = 4; p.ca = 2; p.cb = 2; p.ck = (int)K; p.sh = 0; }
    else if (x8) { p.mul = 2; p.ca = 0; p.cb = 1; p.ck = 0; p.sh = 7 - bits_w; }   // 2 sum v_x op_w + sum op_w
    else { p.mul = 2; p.ca = 1; p.cb = 0; p.ck = 0; p.sh = 7 - bits_x; }
    p.rs_a = p.ca ? rs_a : nullptr;                      // row sums of the x operand bytes
    p.rs_b = p.cb ? rs_b : nullptr;                      // row sums of the w operand bytes
    p.y = y; p.y_dtype = y_dtype; p.ldy = ldy; p.acc = acc; p.mask = nullptr; p.sw2 = nullptr; p.up_row0 = 0;
    p.status = device_status_word();
    if (!p.status) return QUEST_ERR_CUDA;

    const bool wide = N > 128;
    const bool pair = wide && M > 128;             // 256 x 256 tiles on CTA pairs
    CUtensorMap tmA, tmB;
    int s = make_operand_map(&tmA, a8, M, K, BM);
    if (s) return s;
    s = make_operand_map(&tmB, b8, N, K, pair ? 128 : wide ? 256 : 128);
    if (s) return s;
    const bool corr = (bits_x == 8) || (bits_w == 8);
    // y through TMA tile stores when its base and row pitch allow it (16-byte multiples)
    const size_t esz = y_dtype == QUEST_F32 ? 4 : 2;
    const bool yt = y && (reinterpret_cast<uintptr_t>(y) % 16 == 0) && ((size_t)ldy * esz % 16 == 0);
    CUtensorMap tmY = tmA;                               // placeholder when unused
    if (yt) {
        s = make_output_map(&tmY, y, M, (int64_t)N * (int64_t)esz, (int64_t)ldy * (int64_t)esz);
        if (s) return s;
    }
#define QUEST_GEMM(BNV, TWOV)                                                                        \
    (corr ? (yt ? launch_gemm_bn<BNV, 1, TWOV, true>(tmA, tmB, tmY, p, st)                            \
                : launch_gemm_bn<BNV, 1, TWOV, false>(tmA, tmB, tmY, p, st))                           \
          : (yt ? launch_gemm_bn<BNV, 0, TWOV, true>(tmA, tmB, tmY, p, st)                            \
                : launch_gemm_bn<BNV, 0, TWOV, false>(tmA, tmB, tmY, p, st)))
    if (pair && !corr && yt && y_dtype == QUEST_BF16 && !acc) {
        // at most two tiles per CTA pair: the form that hides the cluster barriers of set-up and exit
        int dev = 0, sms = 148;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int64_t tiles = ((M + 255) / 256) * ((N + 255) / 256);
        if (tiles <= 2 * (int64_t)(sms / 2)) return launch_gemm_bn<256, 0, true, true, 0, false, true>(tmA, tmB, tmY, p, st);
    }
    if (pair) return QUEST_GEMM(256, true);
    if (wide) return QUEST_GEMM(256, false);
    return QUEST_GEMM(128, false);
#undef QUEST_GEMM
}

// Gate and up projections of an MLP block with the SwiGLU fused into the epilogue:
//   h[i][j] = bf16( silu(sx[i] sw_gate[j] acc_g[i][j]) * (sx[i] sw_up[j] acc_u[i][j]) ),  j < I,
// where b8 stacks the operand rows of w_gate ([0, I)) and w_up ([I, 2I)) and rs_b their row sums.
int launch_gemm_swiglu(const int8_t *a8, const int8_t *b8, const int32_t *rs_a, const int32_t *rs_b, int bits,
                       const float *sx, const float *sw_gate, const float *sw_up, int64_t M, int64_t I, int64_t K,
                       void *h, cudaStream_t st) {
    if (M == 0 || I == 0) return QUEST_OK;
    const bool mx = e2m1_operands(bits, bits), b8x = bits == 8;
    GemmParams p;
    p.M = (int)M; p.N = (int)I; p.K = (int)(mx ? K / 2 : K);
    p.sx = sx; p.sw = sw_gate; p.sw2 = sw_up; p.up_row0 = (int)I;
    if (mx) { p.mul = 1; p.ca = 0; p.cb = 0; p.ck = 0; p.sh = 0; }
    else if (b8x) { p.mul = 4; p.ca = 2; p.cb = 2; p.ck = (int)K; p.sh = 0; }
    else { p.mul = 1; p.ca = 0; p.cb = 0; p.ck = 0; p.sh = 14 - 2 * bits; }
    p.rs_a = b8x ? rs_a : nullptr; p.rs_b = b8x ? rs_b : nullptr;
    p.y = h; p.y_dtype = QUEST_BF16; p.ldy = I; p.acc = nullptr; p.mask = nullptr;
    p.status = device_status_word();
    if (!p.status) return QUEST_ERR_CUDA;
    const bool pair = M > 128;
    CUtensorMap tmA, tmB, tmY;
    int s = make_operand_map(&tmA, a8, M, p.K, BM);
    if (s) return s;
    if ((s = make_operand_map(&tmB, b8, 2 * I, p.K, 128))) return s;       // boxes of 128 rows: gate rows or up rows
    if ((s = make_output_map(&tmY, h, M, I * 2, I * 2))) return s;
#define QUEST_GEMM_SG(MODEV) \
    (pair ? launch_gemm_bn<256, MODEV, true, true, 0, true>(tmA, tmB, tmY, p, st) \
          : launch_gemm_bn<256, MODEV, false, true, 0, true>(tmA, tmB, tmY, p, st))
    if (mx) return QUEST_GEMM_SG(5);
    if (b8x) return QUEST_GEMM_SG(1);
    return QUEST_GEMM_SG(0);
#undef QUEST_GEMM_SG
}

// Backward-pass contraction (the two products of Algorithm 2): out[i][j] = mask[i][j] * sum_k A(i, k) B(j, k) with
// bfloat16 operands and binary32 output [I x J].  `opl` says how the operands lie in memory:
//   0: a [I x Kc], b [J x Kc], the contraction index contiguous (K-major);
//   1: a [I x Kc] K-major, b [Kc x J] (memory rows run along the contraction: MN-major);
//   2: a [Kc x I] and b [Kc x J], both MN-major.
// With fuse_iht128 (J % 128 == 0, I > 128, J > 128) the epilogue also applies the inverse Hadamard
// transform on blocks of 128 columns and stores out_dtype; otherwise out is binary32.
int launch_gemm_bf16_masked(const void *a, const void *b, int64_t I, int64_t J, int64_t Kc,
                            const uint8_t *mask, void *out, int out_dtype, bool fuse_iht128, int opl, cudaStream_t st) {
    if (I == 0 || J == 0) return QUEST_OK;
    GemmParams p;
    p.M = (int)I; p.N = (int)J; p.K = (int)(2 * Kc);
    p.sx = nullptr; p.sw = nullptr; p.rs_a = nullptr; p.rs_b = nullptr;
    p.mul = 1; p.ca = 0; p.cb = 0; p.ck = 0; p.sh = 0;
    p.y = out; p.y_dtype = out_dtype; p.ldy = J; p.acc = nullptr; p.mask = mask; p.sw2 = nullptr; p.up_row0 = 0;
    const int64_t esz = out_dtype == QUEST_F32 ? 4 : 2;
    p.status = device_status_word();
    if (!p.status) return QUEST_ERR_CUDA;
    const bool wide = J > 128;
    const bool pair = wide && I > 128;
    CUtensorMap tmA, tmB, tmY;
    int s;
    // MN-major: the tensor is [Kc rows x I (or J) elements]; a box is 128 bytes of a row x 64 rows
    if (opl == 2) s = make_operand_map(&tmA, reinterpret_cast<const int8_t *>(a), Kc, 2 * I, 64);
    else s = make_operand_map(&tmA, reinterpret_cast<const int8_t *>(a), I, 2 * Kc, BM);
    if (s) return s;
    if (opl >= 1) s = make_operand_map(&tmB, reinterpret_cast<const int8_t *>(b), Kc, 2 * J, 64);
    else s = make_operand_map(&tmB, reinterpret_cast<const int8_t *>(b), J, 2 * Kc, pair ? 128 : wide ? 256 : 128);
    if (s) return s;
    s = make_output_map(&tmY, out, I, J * esz, J * esz);
    if (s) return s;
#define QUEST_GEMM_BWD(BNV, MODEV, TWOV)                                                  \
    (opl == 2 ? launch_gemm_bn<BNV, MODEV, TWOV, true, 2>(tmA, tmB, tmY, p, st)           \
              : opl == 1 ? launch_gemm_bn<BNV, MODEV, TWOV, true, 1>(tmA, tmB, tmY, p, st) \
                         : launch_gemm_bn<BNV, MODEV, TWOV, true, 0>(tmA, tmB, tmY, p, st))
    if (fuse_iht128) {
        if (!pair || J % 128 != 0) return QUEST_ERR_SHAPE;
        return QUEST_GEMM_BWD(256, 3, true);
    }
    if (out_dtype != QUEST_F32) return QUEST_ERR_DTYPE;
    if (pair) return QUEST_GEMM_BWD(256, 2, true);
    if (wide) return QUEST_GEMM_BWD(256, 2, false);
    return QUEST_GEMM_BWD(128, 2, false);
#undef QUEST_GEMM_BWD
}

// Contraction of E2M1 nibble operands xq [M x K/2], wq [N x K/2] on the FP4 tensor-core path:
// y = sx sw sum_k v_x v_w, acc = acc_mul * sum_k v_x v_w as int32 (the sum is exact in binary32).
int launch_gemm_e2m1(const uint8_t *xq, const uint8_t *wq, const float *sx, const float *sw, int64_t M, int64_t N,
                     int64_t K, void *y, int y_dtype, int64_t ldy, int32_t *acc, int acc_mul, cudaStream_t st) {
    if (M == 0 || N == 0) return QUEST_OK;
    GemmParams p;
    p.M = (int)M; p.N = (int)N; p.K = (int)(K / 2);
    p.sx = sx; p.sw = sw; p.rs_a = nullptr; p.rs_b = nullptr;
    p.mul = acc_mul; p.ca = 0; p.cb = 0; p.ck = 0; p.sh = 0;
    p.y = y; p.y_dtype = y_dtype; p.ldy = ldy; p.acc = acc; p.mask = nullptr; p.sw2 = nullptr; p.up_row0 = 0;
    p.status = device_status_word();
    if (!p.status) return QUEST_ERR_CUDA;
    const bool wide = N > 128;
    const bool pair = wide && M > 128;
    CUtensorMap tmA, tmB;
    int s = make_operand_map(&tmA, reinterpret_cast<const int8_t *>(xq), M, K / 2, BM);
    if (s) return s;
    s = make_operand_map(&tmB, reinterpret_cast<const int8_t *>(wq), N, K / 2, pair ? 128 : wide ? 256 : 128);
    if (s) return s;
    const size_t esz = y_dtype == QUEST_F32 ? 4 : 2;
    const bool yt = y && (reinterpret_cast<uintptr_t>(y) % 16 == 0) && ((size_t)ldy * esz % 16 == 0);
    CUtensorMap tmY = tmA;
    if (yt) {
        s = make_output_map(&tmY, y, M, (int64_t)N * (int64_t)esz, (int64_t)ldy * (int64_t)esz);
        if (s) return s;
    }
#define QUEST_GEMM_MX(BNV, TWOV) \
    (yt ? launch_gemm_bn<BNV, 5, TWOV, true>(tmA, tmB, tmY, p, st) : launch_gemm_bn<BNV, 5, TWOV, false>(tmA, tmB, tmY, p, st))
    if (pair) return QUEST_GEMM_MX(256, true);
    if (wide) return QUEST_GEMM_MX(256, false);
    return QUEST_GEMM_MX(128, false);
#undef QUEST_GEMM_MX
}

int launch_gemm_bf16_scaled(const void *a, const void *b, const float *sw, int64_t M, int64_t N, int64_t K,
                            void *y, int y_dtype, int64_t ldy, cudaStream_t st) {
    if (M == 0 || N == 0) return QUEST_OK;
    GemmParams p;
    p.M = (int)M; p.N = (int)N; p.K = (int)(2 * K);
    p.sx = nullptr; p.sw = sw; p.rs_a = nullptr; p.rs_b = nullptr;
    p.mul = 1; p.ca = 0; p.cb = 0; p.ck = 0; p.sh = 0;
    p.y = y; p.y_dtype = y_dtype; p.ldy = ldy; p.acc = nullptr; p.mask = nullptr; p.sw2 = nullptr; p.up_row0 = 0;
    p.status = device_status_word();
    if (!p.status) return QUEST_ERR_CUDA;
    const bool wide = N > 128;
    const bool pair = wide && M > 128;
    CUtensorMap tmA, tmB;
    int s = make_operand_map(&tmA, reinterpret_cast<const int8_t *>(a), M, 2 * K, BM);
    if (s) return s;
    s = make_operand_map(&tmB, reinterpret_cast<const int8_t *>(b), N, 2 * K, pair ? 128 : wide ? 256 : 128);
    if (s) return s;
    const size_t esz = y_dtype == QUEST_F32 ? 4 : 2;
    const bool yt = (reinterpret_cast<uintptr_t>(y) % 16 == 0) && ((size_t)ldy * esz % 16 == 0);
    CUtensorMap tmY = tmA;
    if (yt) {
        s = make_output_map(&tmY, y, M, (int64_t)N * (int64_t)esz, (int64_t)ldy * (int64_t)esz);
        if (s) return s;
    }
#define QUEST_GEMM_WO(BNV, TWOV) \
    (yt ? launch_gemm_bn<BNV, 4, TWOV, true>(tmA, tmB, tmY, p, st) : launch_gemm_bn<BNV, 4, TWOV, false>(tmA, tmB, tmY, p, st))
    if (pair) return QUEST_GEMM_WO(256, true);
    if (wide) return QUEST_GEMM_WO(256, false);
    return QUEST_GEMM_WO(128, false);
#undef QUEST_GEMM_WO
}

}  // namespace quest
