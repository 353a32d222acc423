// bf16 tensor-core GEMM for sm_100a: tcgen05.mma with TMEM accumulators, TMA-fed operands.
//
// One persistent CTA per SM (192 threads): warp 0 issues TMA loads, warp 1 issues tcgen05.mma and
// owns the TMEM allocation, warps 2..5 run the epilogue (TMEM -> swizzled shared-memory boxes -> bulk
// tensor stores).  Two forms: gemm_kernel, one CTA per 128 x 256 output tile (K step 64, four 48 KiB
// shared-memory stages), and gemm_pair_kernel, clusters of two CTAs sharing one cta_group::2 MMA on a
// 256 x 256 tile (six 32 KiB stages per CTA).  Both keep two accumulator stages in TMEM (2 x 256
// columns) so that the epilogue of tile i overlaps the main loop of tile i+1.
//
// Operands may be K-major (rows of 64 contraction elements = one 128-byte swizzle row) or MN-major
// (the tensor's contiguous dimension is M or N; loaded as 64-wide boxes of 64 contraction rows).
// Several "problems" (up to 3) can share one launch, and a problem's contraction may run over two
// segments with different operand tensors; that is how the MoC contractions are batched:
//   forward   [G | U]          = x  * [Wg ; Wu]^T        two problems, shared A
//   forward   D                = Z' * Wd                 B is MN-major
//   backward  dZ               = dD * Wd^T
//   backward  dWd | dWu | dWg  = Z'^T dD | dU'^T x | dG'^T x    three problems, both operands MN-major
//   backward  dX               = dG' * Wg + dU' * Wu     two contraction segments, B is MN-major
//
// Every wait on an mbarrier is bounded: when the bound expires the kernel raises MOC_ERR_TIMEOUT in
// the device status word, all roles leave their loops, the CTA waits a fixed time for copies in
// flight, frees its TMEM and returns.
#pragma once

#include <cuda.h>

#include "grouped_select.cuh"
#include "moc_common.cuh"

namespace moc {
namespace tc {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4, ACC_STAGES = 2;
constexpr int THREADS = 192;
// the fused 2-of-8 epilogue is arithmetic-heavy: two epilogue warps per TMEM lane quarter there
constexpr int pair_threads(int epi) { return epi == 3 ? 320 : THREADS; }
constexpr uint32_t A_STAGE_BYTES = BM * BK * 2, B_STAGE_BYTES = BN * BK * 2;
constexpr uint32_t STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr uint32_t TMEM_COLS = ACC_STAGES * BN;  // 512
// epilogue staging: per epilogue warp two 32-row x 128-byte boxes (128-byte swizzle atoms, 1024-byte aligned)
constexpr uint32_t EPI_BOX_BYTES = 32 * 128, EPI_BUFS = 2, BAR_REGION_BYTES = 1024;
constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)STAGES * STAGE_BYTES + BAR_REGION_BYTES +
                              4 * EPI_BUFS * EPI_BOX_BYTES;

enum Epilogue : int {
    EPI_F32 = 0,       // C fp32 [M, ldc]
    EPI_GATE_UP = 1,   // problem 0 -> fp32 G [M, ldg]; problem 1 -> bf16 U [M, ldu]
    EPI_BF16 = 2,      // C bf16 [M, ldc]  (optionally accumulating into C)
    // CTA pairs only.  A tile is 256 rows x 128 CHANNELS: the pair's first CTA stages the channels' rows of b_map[0]
    // (W_gate), the second those of b_map[1] (W_up), so the accumulator holds G in columns 0..127 and U in columns
    // 128..255 of the same rows.  The epilogue applies the 2-of-8 mask of MoC 2:8 (Section 4) on the spot and writes
    // the masked hidden state Z' = SiLU(G) . M . U (bf16 [M, ldc], c[0]) and the compact saved triple: no gate or up
    // array ever reaches memory and no selector kernel runs.
    EPI_GATE_UP_2OF8 = 3
};

struct Params {
    CUtensorMap a_map[3];
    CUtensorMap b_map[3];
    int8_t a_idx[3][2];  // [problem][segment] -> tensor map index
    int8_t b_idx[3][2];
    int num_problems;    // 1..3
    int k_segments;      // 1..2
    int k_blocks;        // 64-wide contraction blocks per segment
    int M, N;            // output extent of one problem (rows = A-side, cols = B-side)
    int m_tiles, n_tiles;
    int accumulate;      // EPI_BF16: add the previous content of C
    // outputs
    void *c[3];          // per problem
    int ldc[3];
    CUtensorMap c_map[3];  // per problem: [M, N] with 32-row boxes of 128 bytes (32 fp32 or 64 bf16 columns)
    int direct_store;      // 1: the output cannot be described by a tensor map; threads store their rows
    int single_cta;        // 1: one CTA per tile even where CTA pairs are available (set by the caller)
    // Tile order.  0: (m block, problem, n block) -- tiles of one m block are adjacent, right when the problems share A
    // (gate | up).  1: (problem, m block, n block) -- a wave of CTAs works on ONE problem, right when the problems have
    // different operands on both sides (the three weight gradients: a wave then streams one B matrix instead of two).
    int problem_major;
    // EPI_GATE_UP_2OF8: compact saved activations [M, N / 4] (all three or none)
    int16_t *sv_idx;
    __nv_bfloat16 *sv_g, *sv_u;
    // EPI_GATE_UP_2OF8, when zc != nullptr: Z' leaves in the 2:4-compressed form of the sparse MMA instead of as a
    // dense array -- zc [M, zc_ld] holds the 2 kept (or filler) values of every 4 channels, zmeta the metadata words in
    // the arrangement tensor memory wants ([128-row block][block of 128 channels][row of the block][4 words])
    __nv_bfloat16 *zc;
    int zc_ld;
    uint32_t *zmeta;
    int zmeta_stages;
    int *status;
};

// ---------------------------------------------------------------------------------------------- PTX
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
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
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait (by default about two seconds of SM clock).  Returns false when it gave up or another role already
// did; giving up raises MOC_ERR_TIMEOUT in the device status word and sets *abort_flag.
constexpr long long kWaitLimitCycles = 4000000000LL;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status,
                                          long long limit_cycles = kWaitLimitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3ff) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > limit_cycles) {
                *abort_flag = 1;
                raise_status(status, MOC_ERR_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src),
                 "r"(x), "r"(y)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// 1-D bulk copies: global -> shared (completes on an mbarrier) and shared -> global (bulk group of the thread)
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void bulk_copy_s2g(void *dst, uint32_t src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// the issuing thread's bulk stores: all but the newest `Keep` groups have read their shared-memory source
template <int Keep>
__device__ __forceinline__ void bulk_store_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(Keep) : "memory");
}
__device__ __forceinline__ void bulk_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Programmatic dependent launch: a kernel lets the next kernel of the stream become resident early (its CTAs
// run their set-up and then block in pdl_wait until this grid has completed and its writes are visible).
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap *map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}

// ---- CTA pairs (cta_group::2): one MMA spans the tensor cores, shared memory and TMEM of two CTAs of a cluster
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// tile load whose completion bytes are counted by an mbarrier of the pair's leading CTA (nothing is broadcast: every CTA
// fetches its own boxes)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t leader_bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(leader_bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrives (once the MMAs issued so far have completed) on the barrier at this shared-memory offset in both CTAs
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
        "h"((uint16_t)3)
        : "memory");
}

// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
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
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------- descriptors
// Shared-memory matrix descriptor, 128-byte swizzle, version 1 (sm_100).
//   K-major : rows of 128 bytes, 8-row groups 1024 bytes apart            (LBO unused, SBO = 1024)
//   MN-major: 64-element (128-byte) rows along MN, one row per k; 8 k-rows = 1024 bytes (SBO);
//             the next 64 elements along MN live in the next 64 x BK box (LBO = BK * 128 bytes)
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version
    d |= (uint64_t)2 << 61;  // SWIZZLE_128B
    return d;
}

template <bool A_MN, bool B_MN, int M_INSTR = BM>
__device__ __forceinline__ constexpr uint32_t make_idesc() {
    return (1u << 4)                        // D format: fp32
           | (1u << 7) | (1u << 10)         // A, B format: bf16
           | ((A_MN ? 1u : 0u) << 15) | ((B_MN ? 1u : 0u) << 16)
           | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(M_INSTR >> 4) << 24);
}

// ---------------------------------------------------------------------------------------------- epilogue helpers
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&h);
}

// store 32 consecutive outputs of one row; full vector path when the chunk is inside the row and aligned
__device__ __forceinline__ void store_row_f32(float *dst, const uint32_t (&r)[32], int valid) {
    if (valid >= 32 && ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0)) {
#pragma unroll
        for (int i = 0; i < 8; ++i)
            reinterpret_cast<uint4 *>(dst)[i] = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i < valid) dst[i] = __uint_as_float(r[i]);
    }
}
__device__ __forceinline__ void store_row_bf16(__nv_bfloat16 *dst, const float (&v)[32], int valid) {
    if (valid >= 32 && ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0)) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            reinterpret_cast<uint4 *>(dst)[i] =
                make_uint4(pack_bf16(v[8 * i], v[8 * i + 1]), pack_bf16(v[8 * i + 2], v[8 * i + 3]),
                           pack_bf16(v[8 * i + 4], v[8 * i + 5]), pack_bf16(v[8 * i + 6], v[8 * i + 7]));
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i < valid) dst[i] = __float2bfloat16_rn(v[i]);
    }
}

// ---------------------------------------------------------------------------------------------- epilogue
// One warp moves its 32 rows x BN columns of a finished accumulator (TMEM lanes of the warp, columns at taddr) to
// the output of problem `prob`: rows row0.., columns n0...  warp_boxes: the warp's EPI_BUFS staging boxes.
template <int EPI>
__device__ __forceinline__ void epilogue_tile(const Params &p, int prob, int row0, int n0, uint32_t taddr,
                                              uint32_t warp_boxes, int &ebuf) {
    const int lane = threadIdx.x & 31;
    const int row = row0 + lane;
    const bool row_ok = row < p.M;

    const bool f32_out = EPI == EPI_F32 || (EPI == EPI_GATE_UP && prob == 0);
    const bool direct = p.direct_store != 0 || (EPI == EPI_BF16 && p.accumulate);
    if (direct) {
        // ---- every thread stores its own row (outputs a tensor map cannot describe, accumulation)
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
            uint32_t r[32];
            __syncwarp();
            tmem_ld32(taddr + (uint32_t)c0, r);
            tmem_ld_wait();
            const int col = n0 + c0;
            const int valid = p.N - col;  // columns of this chunk inside the problem
            if (!row_ok || valid <= 0) continue;
            if (f32_out) {
                float *dst = static_cast<float *>(p.c[prob]) + (int64_t)row * p.ldc[prob] + col;
                store_row_f32(dst, r, valid);
            } else {
                __nv_bfloat16 *dst =
                    static_cast<__nv_bfloat16 *>(p.c[prob]) + (int64_t)row * p.ldc[prob] + col;
                float v[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
                if (EPI == EPI_BF16 && p.accumulate) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (i < valid) v[i] += __bfloat162float(dst[i]);
                }
                store_row_bf16(dst, v, valid);
            }
        }
    } else if (row0 < p.M) {
        // ---- 32-row boxes of 128 bytes go through shared memory (thread = row, 16-byte pieces swizzled
        //      the way the tensor map expects) and leave as bulk tensor stores, which clip at M and N
        const uint32_t my_row = (uint32_t)lane * 128u, sw = (uint32_t)(lane & 7);
        if (f32_out) {
#pragma unroll 1
            for (int c0 = 0; c0 < BN && n0 + c0 < p.N; c0 += 32) {
                uint32_t r[32];
                __syncwarp();
                tmem_ld32(taddr + (uint32_t)c0, r);
                tmem_ld_wait();
                if (lane == 0) bulk_store_wait_read<EPI_BUFS - 1>();  // the box about to be refilled is free
                __syncwarp();
                const uint32_t box = warp_boxes + (uint32_t)ebuf * EPI_BOX_BYTES;
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    st_shared_v4(box + my_row + (((uint32_t)i ^ sw) << 4), r[4 * i], r[4 * i + 1], r[4 * i + 2],
                                 r[4 * i + 3]);
                fence_async_smem();
                __syncwarp();
                if (lane == 0) tma_store_2d(&p.c_map[prob], box, n0 + c0, row0);
                ebuf ^= 1;
            }
        } else {
#pragma unroll 1
            for (int c0 = 0; c0 < BN && n0 + c0 < p.N; c0 += 64) {
                uint32_t r[32], q[32];
                __syncwarp();
                tmem_ld32(taddr + (uint32_t)c0, r);
                tmem_ld32(taddr + (uint32_t)c0 + 32u, q);
                tmem_ld_wait();
                if (lane == 0) bulk_store_wait_read<EPI_BUFS - 1>();
                __syncwarp();
                const uint32_t box = warp_boxes + (uint32_t)ebuf * EPI_BOX_BYTES;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    st_shared_v4(box + my_row + (((uint32_t)i ^ sw) << 4),
                                 pack_bf16(__uint_as_float(r[8 * i]), __uint_as_float(r[8 * i + 1])),
                                 pack_bf16(__uint_as_float(r[8 * i + 2]), __uint_as_float(r[8 * i + 3])),
                                 pack_bf16(__uint_as_float(r[8 * i + 4]), __uint_as_float(r[8 * i + 5])),
                                 pack_bf16(__uint_as_float(r[8 * i + 6]), __uint_as_float(r[8 * i + 7])));
                    st_shared_v4(box + my_row + (((uint32_t)(i + 4) ^ sw) << 4),
                                 pack_bf16(__uint_as_float(q[8 * i]), __uint_as_float(q[8 * i + 1])),
                                 pack_bf16(__uint_as_float(q[8 * i + 2]), __uint_as_float(q[8 * i + 3])),
                                 pack_bf16(__uint_as_float(q[8 * i + 4]), __uint_as_float(q[8 * i + 5])),
                                 pack_bf16(__uint_as_float(q[8 * i + 6]), __uint_as_float(q[8 * i + 7])));
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) tma_store_2d(&p.c_map[prob], box, n0 + c0, row0);
                ebuf ^= 1;
            }
        }
    }
}

// Four consecutive bf16 values (w0 = elements 0, 1; w1 = elements 2, 3) with at most two non-zero ones -> the two
// kept values (in order) and the metadata nibble of the sparse MMA: position of the first | position of the second
// << 2, positions ascending; a group with fewer than two non-zero values points its fillers at zero elements.
__device__ __forceinline__ void compress_group4(uint32_t w0, uint32_t w1, uint32_t &packed, uint32_t &nib) {
    const uint32_t e[4] = {w0 & 0xffffu, w0 >> 16, w1 & 0xffffu, w1 >> 16};
    int p0 = -1, p1 = -1;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const bool nz = (e[j] & 0x7fffu) != 0u;
        if (nz && p0 < 0) p0 = j;
        else if (nz && p1 < 0) p1 = j;
    }
    if (p0 < 0) {
        p0 = 0;
        p1 = 1;
    } else if (p1 < 0) {
        p1 = 3;
        if (p0 == 3) p0 = 2;
    }
    uint32_t v0 = 0u, v1 = 0u;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (j == p0) v0 = e[j];
        if (j == p1) v1 = e[j];
    }
    packed = v0 | (v1 << 16);
    nib = (uint32_t)p0 | ((uint32_t)p1 << 2);
}

// Group G8 (channels 8 G8 .. 8 G8 + 7) of a 32-channel chunk: r = gate accumulators, q = up accumulators of one row.
// Writes the group's four words of Z' and its two saved entries (index pair, gate pair, up pair).
template <int G8>
__device__ __forceinline__ void mask_group_2of8(const uint32_t (&r)[32], const uint32_t (&q)[32], uint32_t chunk_channel,
                                                uint32_t (&zw)[16], uint32_t (&iw)[4], uint32_t (&gw)[4],
                                                uint32_t (&uw)[4]) {
    // the two largest gate values by plain float comparison: -0 equals +0 there as in the keys, and NaN is mapped to
    // -inf first; strict comparisons in ascending channel order leave equal values to the lower channel
    float g[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const float v = __uint_as_float(r[8 * G8 + e]);
        g[e] = v != v ? __int_as_float(0xff800000) : v;
    }
    float g1 = g[0], u1 = __uint_as_float(q[8 * G8]);
    int i1 = 0;
#pragma unroll
    for (int e = 1; e < 8; ++e)
        if (g[e] > g1) {
            g1 = g[e];
            u1 = __uint_as_float(q[8 * G8 + e]);
            i1 = e;
        }
    float g2 = 0.f, u2 = 0.f;
    int i2 = -1;
#pragma unroll
    for (int e = 0; e < 8; ++e)
        if (e != i1 && (i2 < 0 || g[e] > g2)) {
            g2 = g[e];
            u2 = __uint_as_float(q[8 * G8 + e]);
            i2 = e;
        }
    const bool swap = i2 < i1;  // saved in ascending channel order
    const int lo = swap ? i2 : i1, hi = swap ? i1 : i2;
    const float glo = swap ? g2 : g1, ghi = swap ? g1 : g2, ulo = swap ? u2 : u1, uhi = swap ? u1 : u2;
    // SiLU(g) = g / (1 + exp(-g)) with the fast exponential and reciprocal (the result is rounded to bf16 anyway);
    // u is rounded to bf16 before the product, as it is where U goes through memory
    const __nv_bfloat16 ub_lo = __float2bfloat16_rn(ulo), ub_hi = __float2bfloat16_rn(uhi);
    const float z_lo = glo * __frcp_rn(1.0f + __expf(-glo)) * __bfloat162float(ub_lo);
    const float z_hi = ghi * __frcp_rn(1.0f + __expf(-ghi)) * __bfloat162float(ub_hi);
    const uint32_t zb_lo = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(z_lo)) << ((lo & 1) * 16);
    const uint32_t zb_hi = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(z_hi)) << ((hi & 1) * 16);
#pragma unroll
    for (int wd = 0; wd < 4; ++wd)
        zw[4 * G8 + wd] = ((lo >> 1) == wd ? zb_lo : 0u) | ((hi >> 1) == wd ? zb_hi : 0u);
    const uint32_t chan = chunk_channel + 8u * G8;
    iw[G8] = (chan + (uint32_t)lo) | ((chan + (uint32_t)hi) << 16);
    gw[G8] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(glo)) |
             ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(ghi)) << 16);
    uw[G8] = (uint32_t)__bfloat16_as_ushort(ub_lo) | ((uint32_t)__bfloat16_as_ushort(ub_hi) << 16);
}

// EPI_GATE_UP_2OF8: one warp's 32 rows x 128 channels of a finished accumulator (G at taddr, U 128 columns further).
// Per group of 8 channels the 2 largest gate values are kept (ties: the lower channel; NaN as -inf); u is rounded to
// bf16 before the product, as it is where U goes through memory, so both forms of the forward agree bit for bit.
__device__ __forceinline__ void epilogue_tile_2of8(const Params &p, int row0, int ch0, int half, uint32_t taddr,
                                                   uint32_t box) {
    // `half`: which 64 channels of the tile this warp takes (two warps share a TMEM lane quarter); box: its staging box
    const int lane = threadIdx.x & 31;
    const int row = row0 + lane;
    const bool row_ok = row < p.M;
    const bool direct = p.direct_store != 0;
    const int K = p.N >> 2;                       // kept channels per row
    const bool vec_saves = (K & 7) == 0;          // 16-byte stores of eight saved entries need 16-byte aligned rows
    const uint32_t my_row = (uint32_t)lane * 128u, sw = (uint32_t)(lane & 7);
    if (row0 >= p.M || ch0 + 64 * half >= p.N) return;
    if (!direct && !p.zc) {
        if (lane == 0) bulk_store_wait_read<0>();  // the previous tile's store has read the box
        __syncwarp();
    }
#pragma unroll 1
    for (int c0 = 64 * half; c0 < 64 * half + 64 && ch0 + c0 < p.N; c0 += 32) {
        uint32_t r[32], q[32];
        __syncwarp();
        tmem_ld32(taddr + (uint32_t)c0, r);
        tmem_ld32(taddr + (uint32_t)(BN / 2 + c0), q);
        tmem_ld_wait();
        uint32_t zw[16];                          // 32 bf16 values of Z'
        uint32_t iw[4], gw[4], uw[4];             // 8 saved entries each
        mask_group_2of8<0>(r, q, (uint32_t)(ch0 + c0), zw, iw, gw, uw);
        mask_group_2of8<1>(r, q, (uint32_t)(ch0 + c0), zw, iw, gw, uw);
        mask_group_2of8<2>(r, q, (uint32_t)(ch0 + c0), zw, iw, gw, uw);
        mask_group_2of8<3>(r, q, (uint32_t)(ch0 + c0), zw, iw, gw, uw);
        const int col = ch0 + c0;
        const int valid = p.N - col;              // channels of this chunk inside the row (a multiple of 8)
        // ---- saved triple: slots (col / 4) .. of the row
        if (p.sv_idx && row_ok) {
            const int64_t o = (int64_t)row * K + (col >> 2);
            if (vec_saves && valid >= 32) {
                *reinterpret_cast<uint4 *>(p.sv_idx + o) = make_uint4(iw[0], iw[1], iw[2], iw[3]);
                *reinterpret_cast<uint4 *>(p.sv_g + o) = make_uint4(gw[0], gw[1], gw[2], gw[3]);
                *reinterpret_cast<uint4 *>(p.sv_u + o) = make_uint4(uw[0], uw[1], uw[2], uw[3]);
            } else {
#pragma unroll
                for (int g8 = 0; g8 < 4; ++g8)
                    if (8 * g8 < valid) {
                        reinterpret_cast<uint32_t *>(p.sv_idx + o)[g8] = iw[g8];
                        reinterpret_cast<uint32_t *>(p.sv_g + o)[g8] = gw[g8];
                        reinterpret_cast<uint32_t *>(p.sv_u + o)[g8] = uw[g8];
                    }
            }
        }
        if (p.zc) {
            // ---- Z' in compressed form: 16 values and one metadata word for the chunk's 32 channels.  The word of a
            // tensor-memory lane joins the 16 bits of two rows eight apart (lane ^ 8), for the chunk's first or second
            // 16 channels: rows with bit 3 clear build the words of the first half, the others those of the second.
            uint32_t pk[8], half16[2] = {0u, 0u};
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                uint32_t nib;
                compress_group4(zw[2 * g], zw[2 * g + 1], pk[g], nib);
                half16[g >> 2] |= nib << (4 * (g & 3));
            }
            const bool upper = (lane & 8) != 0;
            const uint32_t got = __shfl_xor_sync(0xffffffffu, upper ? half16[0] : half16[1], 8);
            const uint32_t word = upper ? (got | (half16[1] << 16)) : (half16[0] | (got << 16));
            const int64_t blk = row0 >> 7;  // row0 is a multiple of 32 inside a 128-row block
            p.zmeta[((blk * p.zmeta_stages + (col >> 7)) * 128 + ((row0 & 127) + lane)) * 4 + ((col >> 5) & 3)] = word;
            if (row_ok) {
                uint4 *dst = reinterpret_cast<uint4 *>(p.zc + (int64_t)row * p.zc_ld + (col >> 1));
                dst[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                dst[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
            }
            continue;
        }
        // ---- Z': the warp's two chunks share one 32-row x 128-byte box
        if (direct) {
            if (row_ok) {
                uint32_t *dst = reinterpret_cast<uint32_t *>(static_cast<__nv_bfloat16 *>(p.c[0]) + (int64_t)row * p.ldc[0] + col);
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    if (2 * i < valid) dst[i] = zw[i];
            }
        } else {
            const int part = (c0 >> 5) & 1;
#pragma unroll
            for (int i = 0; i < 4; ++i)
                st_shared_v4(box + my_row + (((uint32_t)(4 * part + i) ^ sw) << 4), zw[4 * i], zw[4 * i + 1], zw[4 * i + 2],
                             zw[4 * i + 3]);
            if (part == 1 || ch0 + c0 + 32 >= p.N) {  // (a lone first part at the end of the row: the rest is clipped away)
                fence_async_smem();
                __syncwarp();
                if (lane == 0) tma_store_2d(&p.c_map[0], box, ch0 + 64 * half, row0);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------- kernel
template <bool A_MN, bool B_MN, int EPI>
__global__ void __launch_bounds__(THREADS, 1) gemm_kernel(const __grid_constant__ Params p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // 128-byte swizzle atoms need 1024-byte alignment
    uint8_t *smem = smem_raw + (base - raw);
    const uint32_t bar_base = base + STAGES * STAGE_BYTES;
    const uint32_t epi_base = bar_base + BAR_REGION_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + ACC_STAGES + a); };
    volatile uint32_t *tmem_holder =
        reinterpret_cast<volatile uint32_t *>(smem + STAGES * STAGE_BYTES + 8 * (2 * STAGES + 2 * ACC_STAGES));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_per_problem = p.m_tiles * p.n_tiles;
    const int total_tiles = tiles_per_problem * p.num_problems;
    const int kb_total = p.k_blocks * p.k_segments;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < ACC_STAGES; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), 4);  // one arrival per epilogue warp
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_holder)), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    // tile id -> (m block, problem, n block): all tiles of one m block are adjacent, so CTAs running at
    // the same time share A rows and the (small) B operands stay in L2
    auto decode_tile = [&](int tile, int &m_blk, int &prob, int &n_blk) {
        if (p.problem_major) {
            prob = tile / tiles_per_problem;
            const int r = tile - prob * tiles_per_problem;
            m_blk = r / p.n_tiles;
            n_blk = r - m_blk * p.n_tiles;
            return;
        }
        const int per_m = p.num_problems * p.n_tiles;
        m_blk = tile / per_m;
        const int r = tile - m_blk * per_m;
        prob = r / p.n_tiles;
        n_blk = r - prob * p.n_tiles;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            for (int i = 0; i < 3; ++i) {
                prefetch_tmap(&p.a_map[i]);
                prefetch_tmap(&p.b_map[i]);
            }
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                int m_blk, prob, n_blk;
                decode_tile(tile, m_blk, prob, n_blk);
                for (int kb = 0; kb < kb_total; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    const int seg = kb / p.k_blocks, kk = (kb - seg * p.k_blocks) * BK;
                    const CUtensorMap *am = &p.a_map[p.a_idx[prob][seg]];
                    const CUtensorMap *bm = &p.b_map[p.b_idx[prob][seg]];
                    const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
                    mbar_expect_tx(full_bar(stage), STAGE_BYTES);
                    if (A_MN) {
#pragma unroll
                        for (int i = 0; i < BM / 64; ++i)
                            tma_load_2d(sa + i * (64 * BK * 2), am, full_bar(stage), m_blk * BM + i * 64, kk);
                    } else {
                        tma_load_2d(sa, am, full_bar(stage), kk, m_blk * BM);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int i = 0; i < BN / 64; ++i)
                            tma_load_2d(sb + i * (64 * BK * 2), bm, full_bar(stage), n_blk * BN + i * 64, kk);
                    } else {
                        tma_load_2d(sb, bm, full_bar(stage), kk, n_blk * BN);
                    }
                    if (++stage == STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc<A_MN, B_MN>();
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status)) break;
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)acc * BN;
                for (int kb = 0; kb < kb_total; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        // one instruction consumes 16 contraction elements: 32 bytes along a K-major row,
                        // or 16 rows of 128 bytes in an MN-major box
                        const uint64_t ad = A_MN ? make_smem_desc(sa + k * 2048, BK * 128, 1024)
                                                 : make_smem_desc(sa + k * 32, 16, 1024);
                        const uint64_t bd = B_MN ? make_smem_desc(sb + k * 2048, BK * 128, 1024)
                                                 : make_smem_desc(sb + k * 32, 16, 1024);
                        umma_bf16(tmem_d, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    umma_commit(empty_bar(stage));  // frees the stage once these MMAs have read it
                    if (++stage == STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                umma_commit(tfull_bar(acc));  // accumulator complete
                if (++acc == ACC_STAGES) {
                    acc = 0;
                    acc_phase ^= 1u;
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int quarter = warp & 3;  // TMEM lanes 32*quarter .. +31 are the ones this warp may read
        int acc = 0, ebuf = 0;
        uint32_t acc_phase = 0;
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
            int m_blk, prob, n_blk;
            decode_tile(tile, m_blk, prob, n_blk);
            // the whole warp must agree: the TMEM loads below are warp-collective
            if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status))) break;
            tc_fence_after();
            epilogue_tile<EPI>(p, prob, m_blk * BM + quarter * 32, n_blk * BN,
                               tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * BN,
                               epi_base + (uint32_t)quarter * EPI_BUFS * EPI_BOX_BYTES, ebuf);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
            if (++acc == ACC_STAGES) {
                acc = 0;
                acc_phase ^= 1u;
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    if (warp >= 2 && lane == 0) bulk_store_wait_all();  // shared memory must outlive the stores that read it
    if (*abort_flag) {
        // give copies and MMAs still in flight time to land before shared memory and TMEM go away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}


// ---------------------------------------------------------------------------------------------- pair kernel
// The same GEMM with the CTAs working in pairs (clusters of two, `cta_group::2`): a pair owns a 256 x 256 output
// tile; each CTA stages its own 128 rows of A and HALF of the B tile (128 of the 256 columns), and one
// `tcgen05.mma.cta_group::2` issued by the pair's leading CTA multiplies both A halves with both B halves, each
// CTA's TMEM receiving its 128 rows.  Per CTA and k-block that is 32 KiB of operands instead of 48 KiB: a third
// less traffic from L2 and a six-deep ring in the same shared memory.
//   full[s]   (leader's)  : counts the bytes both CTAs' loads bring in for stage s
//   empty[s]  (each CTA's): the leader's commit arrives on it in both CTAs when the MMAs have read stage s
//   tfull[a]  (each CTA's): ... when accumulator a is complete
//   tempty[a] (leader's)  : the eight epilogue warps of the pair arrive when they have drained accumulator a
constexpr int PAIR_STAGES = 6;
constexpr uint32_t PAIR_B_STAGE_BYTES = (BN / 2) * BK * 2, PAIR_STAGE_BYTES = A_STAGE_BYTES + PAIR_B_STAGE_BYTES;
static_assert(PAIR_STAGES * PAIR_STAGE_BYTES == STAGES * STAGE_BYTES, "both kernels use the same shared-memory layout");

template <bool A_MN, bool B_MN, int EPI>
__global__ void __launch_bounds__(pair_threads(EPI), 1) gemm_pair_kernel(const __grid_constant__ Params p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // 128-byte swizzle atoms need 1024-byte alignment
    uint8_t *smem = smem_raw + (base - raw);
    const uint32_t bar_base = base + PAIR_STAGES * PAIR_STAGE_BYTES;
    const uint32_t epi_base = bar_base + BAR_REGION_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (PAIR_STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * PAIR_STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * PAIR_STAGES + ACC_STAGES + a); };
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(
        smem + PAIR_STAGES * PAIR_STAGE_BYTES + 8 * (2 * PAIR_STAGES + 2 * ACC_STAGES));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();  // 0: the pair's leading CTA
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int m_pairs = (p.m_tiles + 1) >> 1;  // 256-row blocks
    const int total_tiles = m_pairs * p.n_tiles * p.num_problems;
    const int kb_total = p.k_blocks * p.k_segments;

    if (threadIdx.x == 0) {
        for (int s = 0; s < PAIR_STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < ACC_STAGES; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), 2 * (pair_threads(EPI) / 32 - 2));  // one arrival per epilogue warp of the pair
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(const_cast<uint32_t *>(tmem_holder)), TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the partner's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    auto decode_tile = [&](int tile, int &m_blk, int &prob, int &n_blk) {
        const int per_m = p.num_problems * p.n_tiles;
        m_blk = tile / per_m;
        const int r = tile - m_blk * per_m;
        prob = r / p.n_tiles;
        n_blk = r - prob * p.n_tiles;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (one per CTA)
        if (lane == 0) {
            for (int i = 0; i < 3; ++i) {
                prefetch_tmap(&p.a_map[i]);
                prefetch_tmap(&p.b_map[i]);
            }
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = pair; tile < total_tiles && ok; tile += num_pairs) {
                int m_blk, prob, n_blk;
                decode_tile(tile, m_blk, prob, n_blk);
                const int m0 = m_blk * (2 * BM) + (int)rank * BM;          // this CTA's rows of A
                // this CTA's half of the B tile (EPI_GATE_UP_2OF8: the same channels of its own weight matrix)
                const int nb0 = EPI == EPI_GATE_UP_2OF8 ? n_blk * (BN / 2) : n_blk * BN + (int)rank * (BN / 2);
                for (int kb = 0; kb < kb_total; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    const int seg = kb / p.k_blocks, kk = (kb - seg * p.k_blocks) * BK;
                    const CUtensorMap *am = &p.a_map[p.a_idx[prob][seg]];
                    const CUtensorMap *bm = &p.b_map[EPI == EPI_GATE_UP_2OF8 ? (int)rank : p.b_idx[prob][seg]];
                    const uint32_t sa = base + stage * PAIR_STAGE_BYTES, sb = sa + A_STAGE_BYTES;
                    const uint32_t lead_full = map_to_cta(full_bar(stage), 0);
                    if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * PAIR_STAGE_BYTES);
                    if (A_MN) {
#pragma unroll
                        for (int i = 0; i < BM / 64; ++i)
                            tma_load_2d_pair(sa + i * (64 * BK * 2), am, lead_full, m0 + i * 64, kk);
                    } else {
                        tma_load_2d_pair(sa, am, lead_full, kk, m0);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int i = 0; i < BN / 128; ++i)
                            tma_load_2d_pair(sb + i * (64 * BK * 2), bm, lead_full, nb0 + i * 64, kk);
                    } else {
                        tma_load_2d_pair(sb, bm, lead_full, kk, nb0);
                    }
                    if (++stage == PAIR_STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leading CTA only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = make_idesc<A_MN, B_MN, 2 * BM>();
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = pair; tile < total_tiles && ok; tile += num_pairs) {
                if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status)) break;
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)acc * BN;
                for (int kb = 0; kb < kb_total; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = base + stage * PAIR_STAGE_BYTES, sb = sa + A_STAGE_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        const uint64_t ad = A_MN ? make_smem_desc(sa + k * 2048, BK * 128, 1024)
                                                 : make_smem_desc(sa + k * 32, 16, 1024);
                        const uint64_t bd = B_MN ? make_smem_desc(sb + k * 2048, BK * 128, 1024)
                                                 : make_smem_desc(sb + k * 32, 16, 1024);
                        umma_bf16_pair(tmem_d, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    umma_commit_pair(empty_bar(stage));  // frees the stage in both CTAs
                    if (++stage == PAIR_STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                umma_commit_pair(tfull_bar(acc));  // accumulator complete, in both CTAs
                if (++acc == ACC_STAGES) {
                    acc = 0;
                    acc_phase ^= 1u;
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5 of each CTA)
        const int quarter = warp & 3;
        int acc = 0, ebuf = 0;
        uint32_t acc_phase = 0;
        for (int tile = pair; tile < total_tiles; tile += num_pairs) {
            int m_blk, prob, n_blk;
            decode_tile(tile, m_blk, prob, n_blk);
            if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status))) break;
            tc_fence_after();
            if (EPI == EPI_GATE_UP_2OF8)
                epilogue_tile_2of8(p, m_blk * (2 * BM) + (int)rank * BM + quarter * 32, n_blk * (BN / 2), (warp - 2) >> 2,
                                   tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * BN,
                                   epi_base + (uint32_t)(warp - 2) * EPI_BOX_BYTES);
            else
                epilogue_tile<EPI>(p, prob, m_blk * (2 * BM) + (int)rank * BM + quarter * 32, n_blk * BN,
                                   tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * BN,
                                   epi_base + (uint32_t)quarter * EPI_BUFS * EPI_BOX_BYTES, ebuf);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));
            if (++acc == ACC_STAGES) {
                acc = 0;
                acc_phase ^= 1u;
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    if (warp >= 2 && lane == 0) bulk_store_wait_all();  // shared memory must outlive the stores that read it
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // neither CTA leaves while the partner may still read its shared memory or signal it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

// ---------------------------------------------------------------------------------------------- wait probe
// One warp waits, with the bounded wait every kernel here uses, on an mbarrier that nothing ever completes.  The
// wait runs out after `limit_cycles`, raises MOC_ERR_TIMEOUT and the kernel returns normally: the test of the
// time-out path (nothing traps, faults or spins without end).
__global__ void bounded_wait_probe_kernel(long long limit_cycles, int *status, int *gave_up) {
    __shared__ uint64_t bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const bool ok = mbar_wait(smem_u32(&bar), 0, &s_abort, status, limit_cycles);
    if (threadIdx.x == 0 && gave_up) *gave_up = ok ? 0 : 1;
}

}  // namespace tc
}  // namespace moc
