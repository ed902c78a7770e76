// CFI_VARIANT_DENSE_TC for bf16 layers at very large batch: a persistent kernel with 128 x 256 tiles.
//
// Included by cfi_layer.cu after cfi_dense_tc.cuh (same operands and helpers).
//
// Two things hold the one-tile kernel (128 x 128 tiles, two CTAs per SM) back at 50,432 rows.  One thread gets an
// MMA instruction accepted only about every 150 cycles whatever its N (measured with a stand-alone loop), so N = 128
// leaves tensor throughput on the table that N = 256 gets.  And the epilogue of one tile overlaps the main loop of
// another only by chance: CTAs that start together stay in step, contend for the tensor pipe during their main
// loops and for the ALUs during their epilogues; for the 768 -> 3072 layer with GELU the epilogue costs about as
// much as the tile's twelve K blocks.  Here one CTA per SM walks over many 128 x 256 tiles and the overlap is built in:
//
//   warp 0, one lane    TMA producer: a 128 x 64 box of x and a 256 x 64 box of Wd per K block, for all K blocks of
//                       all this CTA's tiles one after the other through a 4-slot ring of 48 KB slots (the ring
//                       does not drain between tiles);
//   warp 1, one lane    MMA issuer (M = 128, N = 256, K = 16): tile i accumulates into tensor-memory buffer i mod 2
//                       (2 x 256 columns); before reusing a buffer it waits until the epilogue has read it;
//   warps 2..17         epilogue of tile i while the MMAs of tile i + 1 run, in four quarters of 64 columns:
//                       tcgen05.ld (one batch row and 16 columns per thread), bias (read from global memory, the same
//                       64 bytes for a whole warp), activation in packed fp32, bf16, one of two 16 KB staging boxes in
//                       shared memory (128-byte swizzle), and a TMA store of the box issued by one thread, which
//                       clips rows past the batch and columns past out.  While the store of one box drains, the
//                       next quarter is computed into the other; the issuing thread waits for a box's store to have
//                       read shared memory (cp.async.bulk.wait_group.read) one barrier before the box is written again.
//
// Tiles are numbered with the output tile fastest, and CTA c takes tiles c, c + gridDim.x, ...: CTAs running at the
// same time share a batch tile of x, and Wd (4.7 MB for 768 x 3072) stays in L2.
//
// Barriers: full/empty per ring slot as in the one-tile kernel, with the phase taken from a running count of K
// blocks; acc_full[b] (tcgen05.commit after a tile's last MMA) and acc_empty[b] (one arrival per epilogue warp once
// its tcgen05.ld of the tile have completed).  Every wait is bounded (status code 2); a role that gives up leaves
// its loop, the roles waiting on it give up in turn, and all meet at the final barrier; there the CTA waits (bounded) for
// the boxes still on their way into its shared memory and for its last MMA, then frees tensor memory and ends.

constexpr int kTpN = 256, kTpStages = 4, kTpEpilogueWarps = 16, kTpThreads = 64 + 32 * kTpEpilogueWarps;
constexpr uint32_t kTpABytes = kTcM * kTcK * 2, kTpBBytes = kTpN * kTcK * 2, kTpStageBytes = kTpABytes + kTpBBytes;  // 16 + 32 KB
constexpr uint32_t kTpStoreBoxBytes = kTcM * 64 * 2;       // one TMA store box of y: 128 rows x 64 bf16 = 16 KB
constexpr uint32_t kTpStagingBytes = 2 * kTpStoreBoxBytes;  // two boxes, written and stored alternately
constexpr size_t kTpSmemBytes = 1024 + kTpStages * kTpStageBytes + kTpStagingBytes + 2048;  // exactly 227 KB
constexpr uint32_t kTpTmemCols = 512;
constexpr uint32_t kTpInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTpN >> 3) << 17) | ((uint32_t)(kTcM >> 4) << 24);

__device__ __forceinline__ void umma_bf16_n256(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}" ::"r"(tmem_d),
        "l"(desc_a), "l"(desc_b), "r"(kTpInstrDesc), "r"(accumulate), "r"(0u)
        : "memory");
}

// Shared memory from the first 1024-byte boundary: ring (4 x 48 KB) | two store boxes (2 x 16 KB) | control:
//   +0 full[4], +32 empty[4], +64 acc_full[2], +80 acc_empty[2], +96 tensor-memory base, +104 the issuer's last commit.
template <int ACT>
__global__ void __launch_bounds__(kTpThreads, 1)
cfi_dense_tc_persistent_kernel(DevLayer L, const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                               const __grid_constant__ CUtensorMap map_y, int batch, int n_tiles_n, int n_tiles) {
    pdl_launch_dependents();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t base = ((smem_u32(0) + 1023u) & ~1023u) - smem_u32(0);
    const uint32_t ring = base, staging = base + kTpStages * kTpStageBytes, ctl = staging + kTpStagingBytes;
    const uint32_t full0 = smem_u32(ctl), empty0 = smem_u32(ctl + 32), acc_full0 = smem_u32(ctl + 64),
                   acc_empty0 = smem_u32(ctl + 80);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_at(ctl + 96));
    const uint32_t mma_done = smem_u32(ctl + 104);  // the issuer's last commit: every MMA of this CTA has finished
    const int k_blocks = (L.in + kTcK - 1) / kTcK;
    const int first = blockIdx.x, stride = gridDim.x;

    if (tid == 0) {
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_w);
        prefetch_tensormap(&map_y);
        for (int s = 0; s < kTpStages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full0 + 8 * b, 1);
            mbar_init(acc_empty0 + 8 * b, kTpEpilogueWarps);
        }
        mbar_init(mma_done, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(ctl + 96)), "r"(kTpTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();  // x and y may belong to the kernel before this one
    bool ok = true;
    uint32_t issued = 0;  // thread 0: K blocks whose boxes it has requested

    if (warp == 0 && lane == 0) {
        // ---------------------------------------------------------------- TMA producer
        uint32_t g = 0;  // K blocks issued so far by this CTA
        for (int t = first; t < n_tiles && ok; t += stride) {
            const int m0 = (t / n_tiles_n) * kTcM, n0 = (t % n_tiles_n) * kTpN;
            for (int kb = 0; kb < k_blocks; ++kb, ++g) {
                const uint32_t s = g % kTpStages, use = g / kTpStages;
                if (use > 0) ok = mbar_wait(empty0 + 8 * s, (use - 1) & 1u, kTcSpinLimit);
                if (!ok) break;
                const uint32_t a_dst = smem_u32(ring + s * kTpStageBytes), b_dst = a_dst + kTpABytes;
                mbar_expect_tx(full0 + 8 * s, kTpStageBytes);
                tma_load_2d(a_dst, &map_x, full0 + 8 * s, kb * kTcK, m0);
                tma_load_2d(b_dst, &map_w, full0 + 8 * s, kb * kTcK, n0);
                issued = g + 1;
            }
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------------------------------------------------------- MMA issuer
        uint32_t g = 0, i = 0;  // K blocks and tiles so far
        for (int t = first; t < n_tiles && ok; t += stride, ++i) {
            const uint32_t b = i & 1u, use = i >> 1;
            if (use > 0) ok = mbar_wait(acc_empty0 + 8 * b, (use - 1) & 1u, kTcSpinLimit);  // the epilogue has read buffer b
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t tmem_d = tmem_base + b * (uint32_t)kTpN;
            for (int kb = 0; kb < k_blocks; ++kb, ++g) {
                const uint32_t s = g % kTpStages;
                ok = mbar_wait(full0 + 8 * s, (g / kTpStages) & 1u, kTcSpinLimit);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_addr = smem_u32(ring + s * kTpStageBytes), b_addr = a_addr + kTpABytes;
                const uint64_t da = umma_desc_k_sw128(a_addr), db = umma_desc_k_sw128(b_addr);
#pragma unroll
                for (int k = 0; k < kTcK / 16; ++k)
                    umma_bf16_n256(tmem_d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), (kb | k) != 0 ? 1u : 0u);
                umma_commit(empty0 + 8 * s);
            }
            if (ok) umma_commit(acc_full0 + 8 * b);  // tile i is complete once every MMA issued so far has finished
        }
        umma_commit(mma_done);
    } else if (warp >= 2) {
        // ---------------------------------------------------------------- epilogue
        const int et = tid - 64;
        const int q = warp & 3;             // tensor-memory lanes 32 q .. 32 q + 31
        const int cq = (warp - 2) >> 2;     // which 16 of a quarter's 64 columns
        const int row = 32 * q + lane;      // batch row of the tile held by this thread
        uint32_t i = 0, step = 0;           // tiles and quarter-tiles so far
        for (int t = first; t < n_tiles; t += stride, ++i) {
            const int m0 = (t / n_tiles_n) * kTcM, n0 = (t % n_tiles_n) * kTpN;
            const uint32_t b = i & 1u;
            if (ok) ok = mbar_wait(acc_full0 + 8 * b, (i >> 1) & 1u, kTcSpinLimit);
            ok = __all_sync(0xffffffffu, ok);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int qs = 0; qs < 4; ++qs, ++step) {
                // Staging buffer step mod 2: one TMA box of 128 rows x 64 bf16 columns in the 128-byte swizzle.  Its
                // last store (two steps ago) was waited for by thread 0 before the barrier of the step in between.
                const uint32_t stage = staging + (step & 1u) * kTpStoreBoxBytes;
                const int c = 64 * qs + 16 * cq;  // column within the tile
                if (ok) {
                    float4 bv[4];  // bias straight from global memory: every lane of a warp reads the same 64 bytes
#pragma unroll
                    for (int e4 = 0; e4 < 4; ++e4) {
                        const int n = n0 + c + 4 * e4;
                        bv[e4] = n < L.out ? __ldg(reinterpret_cast<const float4*>(L.bias + n)) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                    uint32_t v[16];
                    tmem_ld16(tmem_base + ((uint32_t)(32 * q) << 16) + b * (uint32_t)kTpN + (uint32_t)c, v);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    if (qs == 3) {  // the buffer is free for tile i + 2 once every epilogue warp has its values
                        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                        if (lane == 0) mbar_arrive(acc_empty0 + 8 * b);
                    }
                    uint32_t packed[8];
#pragma unroll
                    for (int e4 = 0; e4 < 4; ++e4) {
                        packed[2 * e4] = bias_act_bf16x2<ACT>(__uint_as_float(v[4 * e4 + 0]), __uint_as_float(v[4 * e4 + 1]), bv[e4].x, bv[e4].y);
                        packed[2 * e4 + 1] = bias_act_bf16x2<ACT>(__uint_as_float(v[4 * e4 + 2]), __uint_as_float(v[4 * e4 + 3]), bv[e4].z, bv[e4].w);
                    }
                    const int ch = 2 * cq;  // 16-byte chunk of the row's 128 bytes; chunk j sits at j ^ (row & 7)
                    *reinterpret_cast<uint4*>(smem_at(stage + row * 128 + ((ch ^ (row & 7)) << 4))) =
                        make_uint4(packed[0], packed[1], packed[2], packed[3]);
                    *reinterpret_cast<uint4*>(smem_at(stage + row * 128 + (((ch + 1) ^ (row & 7)) << 4))) =
                        make_uint4(packed[4], packed[5], packed[6], packed[7]);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the TMA store reads these writes
                }
                if (et == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // the other buffer's store has read it
                asm volatile("bar.sync 1, %0;" ::"n"(32 * kTpEpilogueWarps) : "memory");  // the box is complete
                if (et == 0 && ok && n0 + 64 * qs < L.out) {  // rows past the batch and columns past out are clipped
                    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(
                                     reinterpret_cast<uint64_t>(&map_y)),
                                 "r"(smem_u32(stage)), "r"(n0 + 64 * qs), "r"(m0)
                                 : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
        }
        if (et == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // every store has landed before the CTA ends
    }
    if (!ok) atomicExch(L.status, 2);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    if (__syncthreads_or(!ok)) {
        // A wait gave up somewhere in this CTA.  It must not end while a box is still on its way into its shared memory
        // (the copy would land in, and signal a barrier of, whichever CTA gets that memory next) or while an MMA still
        // works on its tensor memory: wait, again bounded, for the boxes requested and for the issuer's last commit.
        if (tid == 0) {
            for (uint32_t j = issued > (uint32_t)kTpStages ? issued - kTpStages : 0u; j < issued; ++j)
                mbar_wait(full0 + 8 * (j % kTpStages), (j / kTpStages) & 1u, kTcSpinLimit);
            mbar_wait(mma_done, 0u, kTcSpinLimit);
        }
        __syncthreads();
    }
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTpTmemCols) : "memory");
    }
}
