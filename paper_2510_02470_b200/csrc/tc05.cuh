// Thin wrappers over the sm_100a instructions the tensor-core kernels use: mbarrier, TMA tile loads
// (cp.async.bulk.tensor, never multicast), tcgen05 (TMEM allocation, MMA, commit, TMEM loads) and the
// shared-memory / instruction descriptors of the 128-byte-swizzled operand layouts.
//
// Every wait is bounded: a wait that runs out raises a block-wide abort flag, every role leaves its
// loop, the block frees its TMEM and returns, and the host reads an error word.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sage {
namespace tc {

constexpr long long kWaitLimitCycles = 4000000000ll;   // about two seconds at 1.9 GHz

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

// ---- mbarrier ------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Waits for the phase with the given parity to complete. Returns false (and raises *abort) when the limit
// runs out or when another thread of the block has already given up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*abort) return false;
        if (clock64() - t0 > kWaitLimitCycles) {
            *abort = 1;
            return false;
        }
    }
    return true;
}
// Bounded wait that raises nothing (used on the way out of a block).
__device__ __forceinline__ void mbar_wait_quiet(uint64_t* bar, uint32_t parity, long long limit_cycles) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity) && clock64() - t0 < limit_cycles) {}
}

// ---- TMA -----------------------------------------------------------------------------------------
// 2-D tile load; x is the innermost (contiguous) coordinate in elements and must make x * element size a
// multiple of 16 bytes; y is the row. Completion is signalled on the mbarrier as transferred bytes.
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* tmap, uint64_t* bar, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(bar)), "r"(x), "r"(y)
                 : "memory");
}
// 4-D tile load (coordinates innermost first; c0 must make c0 * element size a multiple of 16 bytes).
__device__ __forceinline__ void tma_load_4d(void* smem_dst, const CUtensorMap* tmap, uint64_t* bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* tmap) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}
// Makes shared-memory writes of ordinary threads visible to the async proxy (tensor cores, TMA).
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---- tcgen05 -------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {   // whole warp, ncols power of two >= 32
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {        // whole warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, one thread issues. kind::f16 takes both operands as bf16 (or both f16).
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The mbarrier gets one arrival when every MMA issued so far by this thread has finished.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 16 consecutive fp32 columns of this thread's TMEM lane (lane = 32 * (warp % 4) + lane id).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float v[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// The same load without the wait, for several loads in flight: the registers hold the data only after
// tmem_ld_wait() AND tmem_ld_use() on them (the latter ties their first use to a point after the wait).
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t r[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_use(uint32_t r[16]) {
    asm volatile("" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]), "+r"(r[9]),
                      "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
                 :
                 : "memory");
}

// ---- descriptors ---------------------------------------------------------------------------------
// Shared-memory operand descriptor for a tile whose rows are 128 bytes of the contraction index (K-major),
// stored by TMA with the 128-byte swizzle: groups of 8 rows are 1024 bytes apart. The tile base must be
// 1024-byte aligned; stepping along K inside the 128-byte row adds the byte offset to the start address.
// group_stride_bytes: distance between consecutive groups of 8 rows (1024 when the tile is one box of rows x 128 bytes;
// kt * 1024 when a 4-D box interleaved kt K tiles group by group, see make_tmap_4d_ktiles).
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t smem_addr_bytes, uint32_t group_stride_bytes = 1024) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr_bytes & 0x3ffffu) >> 4);   // start address / 16
    d |= static_cast<uint64_t>(1) << 16;                              // leading byte offset (unused for this layout)
    d |= static_cast<uint64_t>(group_stride_bytes >> 4) << 32;        // stride byte offset between groups of 8 rows
    d |= static_cast<uint64_t>(1) << 46;                              // descriptor version of sm_100
    d |= static_cast<uint64_t>(2) << 61;                              // 128-byte swizzle
    return d;
}
// fp32 (tf32) operand tile stored with the NON-contraction index contiguous (MN-major). The tensor cores
// accept such 32-bit operands only in the "128-byte swizzle with 32-byte atoms" layout: one TMA box of
// [k rows][128 bytes] per 128-byte span of the contiguous index, k rows 128 bytes apart, the four 32-byte pieces of
// a row permuted by (row mod 4), so the pattern repeats every 4 k rows = 512 bytes (stride offset); consecutive
// 128-byte spans are `span_bytes` apart (leading offset). One MMA (8 k rows) covers two such groups.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128_atom32(uint32_t smem_addr_bytes, uint32_t span_bytes) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr_bytes & 0x3ffffu) >> 4);
    d |= static_cast<uint64_t>((span_bytes >> 4) & 0x3fffu) << 16;
    d |= static_cast<uint64_t>(512 >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(1) << 61;                              // 128-byte swizzle, 32-byte atoms
    return d;
}
// Instruction descriptor: fp32 accumulate, A and B of one format (1 = bf16, 2 = tf32), M x N tile.
// a_mn / b_mn = 1 when that operand is stored MN-major.
__host__ __device__ inline uint32_t instr_desc(int fmt, int M, int N, int a_mn, int b_mn) {
    return (1u << 4) | (static_cast<uint32_t>(fmt) << 7) | (static_cast<uint32_t>(fmt) << 10) |
           (static_cast<uint32_t>(a_mn) << 15) | (static_cast<uint32_t>(b_mn) << 16) |
           (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}

// ---- host: tensor maps ---------------------------------------------------------------------------
// 2-D row-major tensor (rows x cols elements, row pitch ld elements) -> tile loads of box_rows x 128 bytes
// with the 128-byte swizzle (atom32 != 0: its 32-byte-atom variant, for MN-major fp32 operands). elem_bytes 2
// (bf16) or 4 (fp32). Returns false when TMA's alignment rules do not hold (base 16-byte aligned, pitch a
// multiple of 16 bytes) or the driver refuses.
bool make_tmap_2d(CUtensorMap* out, const void* base, int elem_bytes, uint64_t rows, uint64_t cols, uint64_t ld,
                  uint32_t box_rows, int atom32 = 0);
// Row-major tensor -> boxes of box_rows x box_cols elements WITHOUT swizzle (the box image in shared memory is plain
// row-major); box_cols * elem_bytes must be a multiple of 16.
bool make_tmap_2d_plain(CUtensorMap* out, const void* base, int elem_bytes, uint64_t rows, uint64_t cols, uint64_t ld,
                        uint32_t box_cols, uint32_t box_rows);
// The same row-major tensor seen as 4-D (128 bytes of a row, 8 rows, K tile, group of 8 rows), so that ONE box of
// kt K tiles x box_rows rows reads kt * 128 consecutive bytes at every visit of a row: on rows megabytes apart
// (every row visit a different page) that is what the load rate depends on (measured on 44 MB rows: 4.6 TB/s with
// one K tile per visit, 6.5 TB/s with two, 6.8 TB/s with four). Shared-memory image: [row group][K tile][8 rows][128
// bytes], i.e. K tile t of the box is an operand tile that starts t * 1024 bytes in and whose 8-row groups are
// kt * 1024 bytes apart. Only whole K tiles (cols / (128 / elem_bytes) of them) and whole row groups are
// addressable: rows must be a multiple of 8 (groups past the end read as zero), box_rows a multiple of 8 up to 256.
bool make_tmap_4d_ktiles(CUtensorMap* out, const void* base, int elem_bytes, uint64_t rows, uint64_t cols, uint64_t ld,
                         uint32_t box_rows, uint32_t kt);

}  // namespace tc
}  // namespace sage
