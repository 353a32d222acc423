// 2:4-sparse bf16 tensor-core GEMM for sm_100a: tcgen05.mma.sp with the A operand compressed.
//
// Section 4 ("MoC with structured 2:8 sparsity") keeps 2 of every 8 consecutive channels, so every group of 4
// consecutive channels of the masked hidden state Z' holds at most 2 non-zero values: a row of Z' is a valid 2:4-sparse
// operand of the sparse tensor-core MMA, which contracts over twice as many (logical) channels per instruction as the
// dense one.  The paper leaves this to future work (Section 6.3, "MoC with 2:8 sparsity"); this is it for the down
// projection D = Z' W_down.
//
// Operands
//   A  compressed, K-major: [M, K/2] bf16 -- of every 4 logical contraction elements the 2 kept ones, in order
//   E  metadata: for every kept pair one nibble (position of the first kept element | position of the second << 2,
//      positions 0..3 inside the group of 4), laid out the way tensor memory wants it (see e_word_index below)
//   B  dense, either K-major [N, K] or MN-major [K, N]
// One instruction contracts 32 logical elements: 16 compressed elements of A (32 bytes of a K-major row), 32 of B, and
// one 32-bit column of tensor memory holding the 128 rows' metadata for those 32 elements:
//   lane  = (m % 8) + 8 * (k / 16) + 16 * (m / 16)        m = row of the 128-row tile, k = logical element 0..31
//   bit   = 16 * ((m / 8) % 2) + (k % 16)                  one bit per logical element: 4 bits per group of 4
// Consecutive 32-element blocks use consecutive columns; the instruction takes the even column's address plus the
// column's parity in its descriptor.
//
// Kernel shape: one CTA per 128 x 128 output tile, 128 logical contraction elements per stage (16 KiB of A, 32 KiB of
// B, four metadata columns), four stages; warp 0 issues TMA loads, warp 1 the MMAs, warps 2..5 run the epilogue, warps
// 6..9 bring the stage's metadata from global memory into tensor memory (tcgen05.st: thread = lane).
#pragma once

#include "tc_gemm.cuh"

namespace moc {
namespace tcsp {

using namespace tc;

constexpr int SBM = 128, SBN = 128, SBKL = 128;  // tile; logical contraction elements per stage
constexpr int SSTAGES = 4, SACC = 2;
constexpr int STHREADS = 320;
constexpr uint32_t SA_BYTES = SBM * (SBKL / 2) * 2, SB_BYTES = SBN * SBKL * 2, SSTAGE_BYTES = SA_BYTES + SB_BYTES;
constexpr int ATOMS = SBKL / 32;                 // MMA instructions (metadata columns) per stage
constexpr uint32_t META_COL = SACC * SBN;        // first metadata column
constexpr uint32_t STMEM_COLS = 512;
constexpr size_t SSMEM_BYTES = 1024 + (size_t)SSTAGES * SSTAGE_BYTES + BAR_REGION_BYTES + 4 * EPI_BUFS * EPI_BOX_BYTES;

struct SpParams {
    CUtensorMap a_map;      // compressed A [M, K/2], boxes of 64 x 128 rows
    CUtensorMap b_map;      // B: K-major [N, K] boxes of 64 x 128 rows, or MN-major [K, N] boxes of 64 x 64
    const uint4 *e;         // metadata words [m_tiles][k_stages][128 lanes] x 4 columns
    int k_stages;           // ceil(K / 128)
    int M, N, m_tiles, n_tiles;
    void *c;                // fp32 or bf16 [M, ldc]
    int ldc;
    int out_bf16;
    int *status;
};

__device__ __forceinline__ void umma_sp_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t tmem_e,
                                             uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::1.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(tmem_e), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tmem_st4(uint32_t taddr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};" ::"r"(taddr), "r"(a), "r"(b), "r"(c),
                 "r"(d)
                 : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

template <bool B_MN>
__device__ __forceinline__ constexpr uint32_t make_sp_idesc() {
    return (1u << 2)                        // sparse
           | (1u << 4)                      // D format: fp32
           | (1u << 7) | (1u << 10)         // A, B format: bf16
           | ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(SBN >> 3) << 17) | ((uint32_t)(SBM >> 4) << 24);
}

template <bool B_MN>
__global__ void __launch_bounds__(STHREADS, 1) gemm_sp_kernel(const __grid_constant__ SpParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw);
    const uint32_t bar_base = base + SSTAGES * SSTAGE_BYTES;
    const uint32_t epi_base = bar_base + BAR_REGION_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (SSTAGES + s); };
    auto meta_bar = [&](int s) { return bar_base + 8u * (2 * SSTAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (3 * SSTAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (3 * SSTAGES + SACC + a); };
    volatile uint32_t *tmem_holder =
        reinterpret_cast<volatile uint32_t *>(smem + SSTAGES * SSTAGE_BYTES + 8 * (3 * SSTAGES + 2 * SACC));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = p.m_tiles * p.n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < SSTAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
            mbar_init(meta_bar(s), 4);  // one arrival per metadata warp
        }
        for (int a = 0; a < SACC; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), 4);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_holder)), STMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tmap(&p.a_map);
            prefetch_tmap(&p.b_map);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                const int m_blk = tile / p.n_tiles, n_blk = tile - m_blk * p.n_tiles;
                for (int ks = 0; ks < p.k_stages; ++ks) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    const uint32_t sa = base + stage * SSTAGE_BYTES, sb = sa + SA_BYTES;
                    mbar_expect_tx(full_bar(stage), SSTAGE_BYTES);
                    tma_load_2d(sa, &p.a_map, full_bar(stage), ks * (SBKL / 2), m_blk * SBM);
                    if (B_MN) {
#pragma unroll
                        for (int kb = 0; kb < SBKL / 64; ++kb)
#pragma unroll
                            for (int i = 0; i < SBN / 64; ++i)
                                tma_load_2d(sb + (uint32_t)(kb * (SBN / 64) + i) * (64 * 64 * 2), &p.b_map, full_bar(stage),
                                            n_blk * SBN + i * 64, ks * SBKL + kb * 64);
                    } else {
#pragma unroll
                        for (int kb = 0; kb < SBKL / 64; ++kb)
                            tma_load_2d(sb + (uint32_t)kb * (SBN * 128), &p.b_map, full_bar(stage), ks * SBKL + kb * 64,
                                        n_blk * SBN);
                    }
                    if (++stage == SSTAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc0 = make_sp_idesc<B_MN>();
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status)) break;
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)acc * SBN;
                for (int ks = 0; ks < p.k_stages; ++ks) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status) ||
                        !mbar_wait(meta_bar(stage), phase, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = base + stage * SSTAGE_BYTES, sb = sa + SA_BYTES;
#pragma unroll
                    for (int a = 0; a < ATOMS; ++a) {
                        // 32 logical elements: 32 bytes of A's compressed rows; of B 64 bytes of a K-major row or 32
                        // rows of an MN-major box
                        const uint64_t ad = make_smem_desc(sa + a * 32, 16, 1024);
                        const uint64_t bd =
                            B_MN ? make_smem_desc(sb + (uint32_t)(a >> 1) * ((SBN / 64) * 64 * 64 * 2) + (a & 1) * 4096, 64 * 128, 1024)
                                 : make_smem_desc(sb + (uint32_t)(a >> 1) * (SBN * 128) + (a & 1) * 64, 16, 1024);
                        const uint32_t ecol = META_COL + (uint32_t)(stage * ATOMS + a);
                        umma_sp_bf16(tmem_d, ad, bd, tmem_base + (ecol & ~1u), idesc0 | (ecol & 1u), (ks | a) != 0 ? 1u : 0u);
                    }
                    umma_commit(empty_bar(stage));
                    if (++stage == SSTAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                umma_commit(tfull_bar(acc));
                if (++acc == SACC) {
                    acc = 0;
                    acc_phase ^= 1u;
                }
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int quarter = warp & 3;
        int acc = 0;
        uint32_t acc_phase = 0;
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
            const int m_blk = tile / p.n_tiles, n_blk = tile - m_blk * p.n_tiles;
            if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status))) break;
            tc_fence_after();
            const int row = m_blk * SBM + quarter * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * SBN;
#pragma unroll 1
            for (int c0 = 0; c0 < SBN; c0 += 32) {
                uint32_t r[32];
                __syncwarp();
                tmem_ld32(taddr + (uint32_t)c0, r);
                tmem_ld_wait();
                const int col = n_blk * SBN + c0, valid = p.N - col;
                if (row >= p.M || valid <= 0) continue;
                if (p.out_bf16) {
                    float v[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
                    store_row_bf16(static_cast<__nv_bfloat16 *>(p.c) + (int64_t)row * p.ldc + col, v, valid);
                } else {
                    store_row_f32(static_cast<float *>(p.c) + (int64_t)row * p.ldc + col, r, valid);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
            if (++acc == SACC) {
                acc = 0;
                acc_phase ^= 1u;
            }
        }
    } else {
        // ------------------------------------------------------------------ metadata: global -> tensor memory (warps 6..9)
        const int quarter = warp & 3;  // the TMEM lanes this warp may touch
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
            const int m_blk = tile / p.n_tiles;
            for (int ks = 0; ks < p.k_stages; ++ks) {
                const uint4 w = __ldg(p.e + ((int64_t)m_blk * p.k_stages + ks) * 128 + quarter * 32 + lane);
                if (!__all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status))) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                tmem_st4(tmem_base + ((uint32_t)(quarter * 32) << 16) + META_COL + (uint32_t)(stage * ATOMS), w.x, w.y, w.z, w.w);
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(meta_bar(stage));
                if (++stage == SSTAGES) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
        }
    }

    __syncwarp();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, STMEM_COLS);
    }
}


// ---------------------------------------------------------------------------------------------- pair kernel
// The production form: clusters of two CTAs share one cta_group::2 sparse MMA on a 256 x 256 output tile.  Each CTA
// stages its own 128 rows of compressed A (16 KiB per 128 logical contraction elements), half of the B tile (128 of the
// 256 columns, 32 KiB) and its rows' metadata (2 KiB: the 128 x 16-byte image described above, which is exactly what
// tensor memory wants), all with TMA; the MMA thread copies the metadata into tensor memory (tcgen05.cp, in order with
// the MMAs it issues next) -- bringing it there from registers cost 0.8 us per stage, the whole gain.
// Per instruction a CTA's shared memory delivers 4 KiB of A and 8 KiB of B for 128 clocks of tensor-core work at the
// sparse rate: 96 B/clk, inside the 128 B/clk an SM's shared memory gives (the one-CTA form above needs 192 B/clk).
// What bounds the kernel is the path from L2: 50 KiB per CTA and stage against 32 KiB of the dense kernel for half the
// contraction length.
// Tensor memory: one 256-column accumulator and the metadata ring (4 stages x 4 columns).  There is no room for a second
// accumulator, so the eight epilogue warps first move the whole accumulator into registers (128 columns each) and hand
// it back at once; conversion and stores then overlap the next tile's main loop.
// B is MN-major ([K, N] with N contiguous: the weight matrices of the down projection and of grad_x); the contraction
// may run over two segments (grad_x = dG' Wg + dU' Wu) with their own compressed operands and metadata.
constexpr int PBN = 256;                      // tile columns of the pair
constexpr uint32_t PB_BYTES = (PBN / 2) * SBKL * 2, PE_BYTES = 128 * 16;
constexpr uint32_t PSTAGE_BYTES = SA_BYTES + PB_BYTES + PE_BYTES;  // 16 + 32 + 2 KiB
constexpr int PSTAGES = 4;
constexpr uint32_t PMETA_COL = PBN;           // metadata columns behind the accumulator
constexpr int PTHREADS = 64 + 256;            // TMA, MMA, 8 epilogue warps
constexpr size_t PSMEM_BYTES = 1024 + (size_t)PSTAGES * PSTAGE_BYTES + BAR_REGION_BYTES;

struct SpPairParams {
    CUtensorMap a_map[2];   // per segment: compressed A [M, K/2]
    CUtensorMap b_map[2];   // per segment: B [K, N] (N contiguous), boxes of 64 x 64
    CUtensorMap e_map[2];   // per segment: metadata as [row blocks * k_stages * 128, 4] 32-bit words, boxes of 4 x 128
    int segments, k_stages; // stages of 128 logical contraction elements per segment
    int M, N, m_pairs, n_tiles;
    __nv_bfloat16 *c;       // [M, ldc]
    int ldc;
    int accumulate;         // add the previous content of C (read as bf16) before rounding
    int *status;
};

__device__ __forceinline__ void umma_sp_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t tmem_e,
                                                  uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(tmem_e), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 128 rows x 16 bytes of shared memory (rows contiguous, no swizzle) -> 128 lanes x 4 columns of tensor memory, in both CTAs
__device__ __forceinline__ void tmem_cp_128x128b_pair(uint32_t taddr, uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);
    d |= (uint64_t)(128u >> 4) << 16;  // leading-dimension offset (one 16-byte chunk per row: not used)
    d |= (uint64_t)(128u >> 4) << 32;  // 8 rows of 16 bytes are one 128-byte core matrix; the next follows at once
    d |= (uint64_t)1 << 46;            // descriptor version
    asm volatile("tcgen05.cp.cta_group::2.128x128b [%0], %1;" ::"r"(taddr), "l"(d) : "memory");
}

__global__ void __launch_bounds__(PTHREADS, 1) gemm_sp_pair_kernel(const __grid_constant__ SpPairParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw);
    const uint32_t bar_base = base + PSTAGES * PSTAGE_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (PSTAGES + s); };
    const uint32_t tfull_bar = bar_base + 8u * (2 * PSTAGES), tempty_bar = tfull_bar + 8u;
    volatile uint32_t *tmem_holder =
        reinterpret_cast<volatile uint32_t *>(smem + PSTAGES * PSTAGE_BYTES + 8 * (2 * PSTAGES + 2));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int total_tiles = p.m_pairs * p.n_tiles;
    const int ks_total = p.k_stages * p.segments;

    if (threadIdx.x == 0) {
        for (int s = 0; s < PSTAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        mbar_init(tfull_bar, 1);
        mbar_init(tempty_bar, 16);      // the eight epilogue warps of both CTAs (leader's barrier)
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(const_cast<uint32_t *>(tmem_holder)), STMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (one per CTA)
        if (lane == 0) {
            for (int i = 0; i < 2; ++i) {
                prefetch_tmap(&p.a_map[i]);
                prefetch_tmap(&p.b_map[i]);
                prefetch_tmap(&p.e_map[i]);
            }
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = pair; tile < total_tiles && ok; tile += num_pairs) {
                const int m_blk = tile / p.n_tiles, n_blk = tile - m_blk * p.n_tiles;
                const int m0 = m_blk * (2 * SBM) + (int)rank * SBM;
                const int nb0 = n_blk * PBN + (int)rank * (PBN / 2);
                const int row_block = m_blk * 2 + (int)rank;  // this CTA's 128-row block
                for (int ks = 0; ks < ks_total; ++ks) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    const int seg = ks / p.k_stages, kk = ks - seg * p.k_stages;
                    const uint32_t sa = base + stage * PSTAGE_BYTES, sb = sa + SA_BYTES, se = sb + PB_BYTES;
                    const uint32_t lead_full = map_to_cta(full_bar(stage), 0);
                    if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * PSTAGE_BYTES);
                    tma_load_2d_pair(sa, &p.a_map[seg], lead_full, kk * (SBKL / 2), m0);
                    tma_load_2d_pair(se, &p.e_map[seg], lead_full, 0, (row_block * p.k_stages + kk) * 128);
#pragma unroll
                    for (int kb = 0; kb < SBKL / 64; ++kb)
#pragma unroll
                        for (int i = 0; i < PBN / 128; ++i)
                            tma_load_2d_pair(sb + (uint32_t)(kb * (PBN / 128) + i) * (64 * 64 * 2), &p.b_map[seg], lead_full,
                                             nb0 + i * 64, kk * SBKL + kb * 64);
                    if (++stage == PSTAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leading CTA only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc0 = (1u << 2) | (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) |
                                        ((uint32_t)(PBN >> 3) << 17) | ((uint32_t)((2 * SBM) >> 4) << 24);
            int stage = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = pair; tile < total_tiles && ok; tile += num_pairs) {
                if (!mbar_wait(tempty_bar, acc_phase ^ 1u, abort_flag, p.status)) break;
                tc_fence_after();
                for (int ks = 0; ks < ks_total; ++ks) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = base + stage * PSTAGE_BYTES, sb = sa + SA_BYTES, se = sb + PB_BYTES;
                    const uint32_t ecol0 = PMETA_COL + (uint32_t)(stage * ATOMS);
                    tmem_cp_128x128b_pair(tmem_base + ecol0, se);  // each CTA's metadata into its own tensor memory
#pragma unroll
                    for (int a = 0; a < ATOMS; ++a) {
                        const uint64_t ad = make_smem_desc(sa + a * 32, 16, 1024);
                        const uint64_t bd = make_smem_desc(sb + (uint32_t)(a >> 1) * ((PBN / 128) * 64 * 64 * 2) + (a & 1) * 4096,
                                                           64 * 128, 1024);
                        const uint32_t ecol = ecol0 + (uint32_t)a;
                        umma_sp_bf16_pair(tmem_base, ad, bd, tmem_base + (ecol & ~1u), idesc0 | (ecol & 1u),
                                          (ks | a) != 0 ? 1u : 0u);
                    }
                    umma_commit_pair(empty_bar(stage));
                    if (++stage == PSTAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                umma_commit_pair(tfull_bar);
                acc_phase ^= 1u;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..9 of each CTA)
        const int quarter = warp & 3, half = (warp - 2) >> 2;  // TMEM lanes 32 quarter.., columns 128 half..
        uint32_t acc_phase = 0;
        for (int tile = pair; tile < total_tiles; tile += num_pairs) {
            const int m_blk = tile / p.n_tiles, n_blk = tile - m_blk * p.n_tiles;
            if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar, acc_phase, abort_flag, p.status))) break;
            acc_phase ^= 1u;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(half * 128);
            uint32_t r0[32], r1[32], r2[32], r3[32];
            tmem_ld32(taddr, r0);
            tmem_ld32(taddr + 32u, r1);
            tmem_ld32(taddr + 64u, r2);
            tmem_ld32(taddr + 96u, r3);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar, 0));  // the accumulator may be overwritten
            const int row = m_blk * (2 * SBM) + (int)rank * SBM + quarter * 32 + lane;
            const int n0 = n_blk * PBN + half * 128;
            if (row < p.M) {
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    const uint32_t(&src)[32] = ch == 0 ? r0 : ch == 1 ? r1 : ch == 2 ? r2 : r3;
                    const int col = n0 + ch * 32, valid = p.N - col;
                    if (valid <= 0) break;
                    __nv_bfloat16 *dst = p.c + (int64_t)row * p.ldc + col;
                    float v[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(src[i]);
                    if (p.accumulate) {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (i < valid) v[i] += __bfloat162float(dst[i]);
                    }
                    store_row_bf16(dst, v, valid);
                }
            }
        }
    }

    __syncwarp();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, STMEM_COLS);
    }
}

// ---------------------------------------------------------------------------------------------- compression
// Rows of a dense bf16 array [rows, ld] whose groups of 4 consecutive elements hold at most 2 non-zero values ->
// compressed rows [rows, kc_ld] (2 elements per group: the non-zero ones in order, zero fillers behind or between them so
// that positions stay ascending) and the metadata words in the tensor-memory arrangement.  A group with more than 2
// non-zero values keeps its first 2; the others go to the overflow list (row, column, value) for the caller to treat
// separately (capacity `overflow_cap`; the count keeps counting past it so that the caller can tell).
// One warp per (128-row block, 128-column stage): lane l reads the 4 groups (16 elements) of rows l, l + 32, l + 64, l + 96
// ... simpler: thread = (row of the block, 32-element atom): 128 x 4 threads per block-stage, 512 threads per CTA.
struct Overflow {
    int32_t row;
    int32_t col;
    float value;
};

__global__ void __launch_bounds__(512) compress_2of4_kernel(const __nv_bfloat16 *__restrict__ dense, int64_t rows, int K,
                                                            int ld, __nv_bfloat16 *__restrict__ comp, int kc_ld,
                                                            uint32_t *__restrict__ meta, int k_stages,
                                                            Overflow *__restrict__ overflow, int overflow_cap,
                                                            unsigned int *__restrict__ overflow_n,
                                                            int *__restrict__ bad_status) {
    __shared__ uint32_t s_half[128][4][2];  // [row][atom][k half]: the row's 16 metadata bits for 16 logical elements
    const int r = threadIdx.x & 127, atom = threadIdx.x >> 7;
    const int64_t blocks = (rows + 127) / 128;
    for (int64_t job = blockIdx.x; job < blocks * k_stages; job += gridDim.x) {
        const int64_t blk = job / k_stages;
        const int ks = (int)(job - blk * k_stages);
        const int64_t row = blk * 128 + r;
        const int k0 = ks * 128 + atom * 32;
        uint32_t bits[2] = {0x4444u, 0x4444u};  // filler: positions (0, 1)
        if (row < rows && k0 < K) {
            // 32 logical elements = 64 bytes -> 16 compressed elements = 32 bytes
            uint32_t in[16];
            const uint4 *src = reinterpret_cast<const uint4 *>(dense + row * ld + k0);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint4 v = make_uint4(0, 0, 0, 0);
                if (k0 + 8 * i < K) v = src[i];  // K is a multiple of 8
                in[4 * i] = v.x, in[4 * i + 1] = v.y, in[4 * i + 2] = v.z, in[4 * i + 3] = v.w;
            }
            uint32_t out[8];
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                const uint16_t e[4] = {(uint16_t)(in[2 * g] & 0xffffu), (uint16_t)(in[2 * g] >> 16),
                                       (uint16_t)(in[2 * g + 1] & 0xffffu), (uint16_t)(in[2 * g + 1] >> 16)};
                int p0 = -1, p1 = -1;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool nz = (e[j] & 0x7fffu) != 0;  // +0 and -0 are both "not kept"
                    if (nz) {
                        if (p0 < 0) p0 = j;
                        else if (p1 < 0) p1 = j;
                        else if (bad_status) {
                            raise_status(bad_status, MOC_ERR_BAD_INDEX);  // the caller promised 2:4 rows
                        } else if (overflow) {
                            const unsigned int at = atomicAdd(overflow_n, 1u);
                            if (at < (unsigned int)overflow_cap) {
                                const uint32_t fb = (uint32_t)e[j] << 16;
                                overflow[at] = Overflow{(int32_t)row, k0 + 4 * g + j, __uint_as_float(fb)};
                            }
                        }
                    }
                }
                // two distinct ascending positions; fillers point at zero elements
                if (p0 < 0) {
                    p0 = 0;
                    p1 = 1;
                } else if (p1 < 0) {
                    if (p0 < 3) p1 = 3;
                    else {
                        p1 = 3;
                        p0 = 2;
                    }
                }
                uint16_t v0 = 0, v1 = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (j == p0) v0 = e[j];
                    if (j == p1) v1 = e[j];
                }
                out[g] = (uint32_t)v0 | ((uint32_t)v1 << 16);
                const uint32_t nib = (uint32_t)p0 | ((uint32_t)p1 << 2);
                bits[g >> 2] = (bits[g >> 2] & ~(0xfu << (4 * (g & 3)))) | (nib << (4 * (g & 3)));
            }
            uint4 *dst = reinterpret_cast<uint4 *>(comp + row * kc_ld + (k0 >> 1));
            dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
            dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
        }
        s_half[r][atom][0] = bits[0];
        s_half[r][atom][1] = bits[1];
        __syncthreads();
        // word of lane l, column atom: rows (l % 8) + 16 (l / 16) [bits 0..15] and + 8 [bits 16..31], k half (l / 8) % 2
        {
            const int l = r, kh = (l >> 3) & 1, rr = (l & 7) + 16 * (l >> 4);
            const uint32_t w = (s_half[rr][atom][kh] & 0xffffu) | (s_half[rr + 8][atom][kh] << 16);
            meta[((blk * k_stages + ks) * 128 + l) * 4 + atom] = w;
        }
        __syncthreads();
    }
}

}  // namespace tcsp
}  // namespace moc
