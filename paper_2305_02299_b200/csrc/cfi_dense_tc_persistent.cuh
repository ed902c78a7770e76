// CFI_VARIANT_DENSE_TC for bf16 layers at very large batch: a persistent kernel with 128 x 256 tiles.
//
// Included by cfi_layer.cu after cfi_dense_tc.cuh and cfi_dense_tf32.cuh (same operands and helpers).
//
// Two things hold the one-tile kernel (128 x 128 tiles, two CTAs per SM) back at 50,432 rows.  An MMA instruction has
// a cost that grows slowly with its N (measured on the TF32 kernel: about 50 cycles + 0.43 per column), so N = 128
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
//   warps 2..17         epilogue of tile i while the MMAs of tile i + 1 run, in two halves of 128 columns:
//                       tcgen05.ld (one batch row and 32 columns per thread), bias, activation, bf16, a staging
//                       half-tile in shared memory, 256-byte runs per batch row to y.
//
// Tiles are numbered with the output tile fastest, and CTA c takes tiles c, c + gridDim.x, ...: CTAs running at the
// same time share a batch tile of x, and Wd (4.7 MB for 768 x 3072) stays in L2.
//
// Barriers: full/empty per ring slot as in the one-tile kernel, with the phase taken from a running count of K
// blocks; acc_full[b] (tcgen05.commit after a tile's last MMA) and acc_empty[b] (one arrival per epilogue warp once
// its tcgen05.ld of the tile have completed).  Every wait is bounded (status code 2); a role that gives up leaves
// its loop, the roles waiting on it give up in turn, and all meet at the final barrier where tensor memory is freed.

constexpr int kTpN = 256, kTpStages = 4, kTpEpilogueWarps = 16, kTpThreads = 64 + 32 * kTpEpilogueWarps;
constexpr uint32_t kTpABytes = kTcM * kTcK * 2, kTpBBytes = kTpN * kTcK * 2, kTpStageBytes = kTpABytes + kTpBBytes;  // 16 + 32 KB
constexpr uint32_t kTpStagingBytes = kTcM * 128 * 2;  // half a y tile, bf16: 32 KB
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

// Shared memory from the first 1024-byte boundary: ring (4 x 48 KB) | staging (32 KB) | control:
//   +0 full[4], +32 empty[4], +64 acc_full[2], +80 acc_empty[2], +96 tensor-memory base, +128 bias[256].
template <int ACT>
__global__ void __launch_bounds__(kTpThreads, 1)
cfi_dense_tc_persistent_kernel(DevLayer L, const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                               __nv_bfloat16* __restrict__ y, int batch, int n_tiles_n, int n_tiles) {
    pdl_launch_dependents();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t base = ((smem_u32(0) + 1023u) & ~1023u) - smem_u32(0);
    const uint32_t ring = base, staging = base + kTpStages * kTpStageBytes, ctl = staging + kTpStagingBytes;
    const uint32_t full0 = smem_u32(ctl), empty0 = smem_u32(ctl + 32), acc_full0 = smem_u32(ctl + 64),
                   acc_empty0 = smem_u32(ctl + 80);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_at(ctl + 96));
    float* bias_s = reinterpret_cast<float*>(smem_at(ctl + 128));  // [kTpN], of the tile in the epilogue
    const int k_blocks = (L.in + kTcK - 1) / kTcK;
    const int first = blockIdx.x, stride = gridDim.x;

    if (tid == 0) {
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_w);
        for (int s = 0; s < kTpStages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full0 + 8 * b, 1);
            mbar_init(acc_empty0 + 8 * b, kTpEpilogueWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(ctl + 96)), "r"(kTpTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid >= 64 && tid < 64 + kTpN && first < n_tiles) {  // bias of the first tile
        const int n = (first % n_tiles_n) * kTpN + tid - 64;
        bias_s[tid - 64] = n < L.out ? L.bias[n] : 0.0f;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();  // x and y may belong to the kernel before this one
    bool ok = true;

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
    } else if (warp >= 2) {
        // ---------------------------------------------------------------- epilogue
        const int et = tid - 64;
        const int q = warp & 3;             // tensor-memory lanes 32 q .. 32 q + 31
        const int cq = (warp - 2) >> 2;     // which 32 of a half's 128 columns
        const int row = 32 * q + lane;      // batch row of the tile held by this thread
        uint32_t i = 0;
        for (int t = first; t < n_tiles; t += stride, ++i) {
            const int m0 = (t / n_tiles_n) * kTcM, n0 = (t % n_tiles_n) * kTpN;
            const uint32_t b = i & 1u;
            // Bias of the next tile: requested now, put into bias_s when this tile no longer reads it.
            const int t_next = t + stride;
            float bias_next = 0.0f;
            if (et < kTpN && t_next < n_tiles) {
                const int n = (t_next % n_tiles_n) * kTpN + et;
                bias_next = n < L.out ? L.bias[n] : 0.0f;
            }
            if (ok) ok = mbar_wait(acc_full0 + 8 * b, (i >> 1) & 1u, kTcSpinLimit);
            ok = __all_sync(0xffffffffu, ok);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
            for (int half = 0; half < 2; ++half) {
                if (ok) {
                    // Staging half-tile: 128 rows x 256 bytes, 16-byte chunks permuted by chunk ^ (row & 15).
                    const int c = 32 * cq;  // column within the half
                    uint32_t v[2][16];
                    const uint32_t t_acc =
                        tmem_base + ((uint32_t)(32 * q) << 16) + b * (uint32_t)kTpN + (uint32_t)(128 * half + c);
                    tmem_ld16(t_acc, v[0]);
                    tmem_ld16(t_acc + 16u, v[1]);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    if (half == 1) {  // the buffer is free for tile i + 2 once every epilogue warp has its values
                        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                        if (lane == 0) mbar_arrive(acc_empty0 + 8 * b);
                    }
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        uint32_t packed[8];
#pragma unroll
                        for (int e4 = 0; e4 < 4; ++e4) {
                            const float4 bv = *reinterpret_cast<const float4*>(bias_s + 128 * half + c + 16 * h + 4 * e4);
                            packed[2 * e4] = bias_act_bf16x2<ACT>(__uint_as_float(v[h][4 * e4 + 0]), __uint_as_float(v[h][4 * e4 + 1]), bv.x, bv.y);
                            packed[2 * e4 + 1] = bias_act_bf16x2<ACT>(__uint_as_float(v[h][4 * e4 + 2]), __uint_as_float(v[h][4 * e4 + 3]), bv.z, bv.w);
                        }
                        const int ch = (c + 16 * h) >> 3;
                        *reinterpret_cast<uint4*>(smem_at(staging + row * 256 + ((ch ^ (row & 15)) << 4))) =
                            make_uint4(packed[0], packed[1], packed[2], packed[3]);
                        *reinterpret_cast<uint4*>(smem_at(staging + row * 256 + (((ch + 1) ^ (row & 15)) << 4))) =
                            make_uint4(packed[4], packed[5], packed[6], packed[7]);
                    }
                }
                asm volatile("bar.sync 1, %0;" ::"n"(32 * kTpEpilogueWarps) : "memory");  // staging half-tile complete
                if (ok) {
                    for (int r = et >> 4; r < kTcM; r += 2 * kTpEpilogueWarps) {  // 16 threads per row, 32 rows per pass
                        const int ch = et & 15, m = m0 + r, n = n0 + 128 * half + 8 * ch;
                        if (m < batch && n < L.out) {
                            const uint4 val = *reinterpret_cast<const uint4*>(smem_at(staging + r * 256 + ((ch ^ (r & 15)) << 4)));
                            *reinterpret_cast<uint4*>(y + (size_t)m * L.out + n) = val;
                        }
                    }
                }
                if (half == 1 && et < kTpN) bias_s[et] = bias_next;  // every read of this tile's bias is behind the barrier above
                asm volatile("bar.sync 1, %0;" ::"n"(32 * kTpEpilogueWarps) : "memory");  // staging (and bias) may be rewritten
            }
        }
    }
    if (!ok) atomicExch(L.status, 2);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTpTmemCols) : "memory");
    }
}
