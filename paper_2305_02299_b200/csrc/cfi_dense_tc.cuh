// CFI_VARIANT_DENSE_TC: large batch, bf16 storage, on the tensor cores.
//
// Included by cfi_layer.cu inside its unnamed namespace (it uses DevLayer, activate, smem_at and the
// pdl_* helpers defined there).
//
// The paper notes that a layer trained with SRigL can be run either from the condensed arrays or as a
// dense layer over the kept neurons, with the same weights (Sec. 4.4, last paragraph), and that the dense
// form wins at larger batch.  On B200 this is where that happens: the gather formulation is held to
// about a fifth of the fp32 FMA rate by shared-memory bandwidth, while a dense bf16 contraction on the
// 5th-generation tensor cores is more than twenty times faster than the FMA pipes, so at 90 % sparsity
// ten times the flops still finish several times sooner.  The layer keeps a dense bf16 copy of its
// weight, Wd[out_pad][in] (zero rows for ablated and padding rows), and the forward is
//
//     y[b, o] = act( bias[o] + sum_c x[b, c] * Wd[o, c] )          fp32 accumulation of exact products,
//
// i.e. the same numbers as the condensed forms up to the order of the additions.
//
// One CTA computes a 128 (batch) x 128 (output rows) tile:
//   warp 0, one lane   TMA producer: per 64-column block of x and Wd one 128 x 64 bf16 box each
//                      (cp.async.bulk.tensor, 128-byte swizzle) into a 3-stage ring, completion on mbarriers;
//   warp 1, one lane   issues tcgen05.mma (cta_group::1, kind::f16, M = N = 128, K = 16 per instruction,
//                      both operands K-major from shared memory), accumulator in 128 columns of tensor
//                      memory; tcgen05.commit hands ring slots back and finally signals the epilogue;
//   warps 2..9         epilogue: tcgen05.ld the accumulator (one batch row and half of the 128 columns per
//                      thread), add bias, apply the activation, round to bf16, pass through shared memory
//                      (the drained ring) and write y in 256-byte runs per batch row.
// Two CTAs fit an SM (97 KB of shared memory, 128 of 512 tensor-memory columns each), so one CTA's
// epilogue overlaps the other's main loop.
//
// Every mbarrier wait is bounded.  If one expires the thread records code 2 in the layer's status word and
// leaves its role's loop; all roles still meet at the final barrier, where the CTA waits (bounded) for the boxes
// still on their way into its shared memory and for its last MMA, then frees tensor memory and returns.
//
// With few tiles and a long K the launch may give each tile to a thread-block cluster of up to 8 CTAs (cluster
// dimension z): CTA r contracts the r-th share of the K blocks and leaves its fp32 partial tile (no bias) in its
// shared memory; after the hardware cluster barrier CTA r sums rows [128 r / S, 128 (r + 1) / S) of all S partial
// tiles in rank order through distributed shared memory, adds the bias, applies the activation, rounds to bf16
// and stores; a second cluster barrier keeps every CTA's shared memory alive until its peers have read it.

#include <cuda.h>  // CUtensorMap and the enums of cuTensorMapEncodeTiled (types only; the entry point is looked up at run time)

constexpr int kTcM = 128, kTcN = 128, kTcK = 64, kTcStages = 3;
constexpr int kTcEpilogueWarps = 8, kTcThreads = 64 + 32 * kTcEpilogueWarps;
constexpr uint32_t kTcStageBytes = (kTcM + kTcN) * kTcK * 2;  // 32 KB
constexpr uint32_t kTcSpinLimit = 1u << 22;
constexpr size_t kTcSmemBytes = 1024 + kTcStages * kTcStageBytes + 1024;

__device__ __forceinline__ uint32_t smem_u32(uint32_t off) { return (uint32_t)__cvta_generic_to_shared(smem_at(off)); }

__device__ __forceinline__ void mbar_init(uint32_t mbar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t mbar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(bytes) : "memory");
}
// Returns false if the phase with this parity did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait(uint32_t mbar, uint32_t parity, uint32_t limit) {
    for (uint32_t it = 0; it < limit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(mbar), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void mbar_arrive(uint32_t mbar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(mbar) : "memory");
}
// Asks for a tensor map's 128 bytes ahead of the first TMA that uses it.
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t mbar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(mbar), "r"(c0), "r"(c1)
        : "memory");
}

// Asks for one box of a tensor map to be brought into L2; nothing is read into the SM.
__device__ __forceinline__ void tma_prefetch_l2_2d(const CUtensorMap* map, int c0, int c1) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1)
                 : "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile stored as rows of 128 bytes with the 128-byte
// swizzle (what the TMA box above produces): groups of 8 rows are 1024 bytes apart (stride offset), the
// leading offset is not used by swizzled K-major layouts, descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t umma_desc_k_sw128(uint32_t smem_addr_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr_bytes & 0x3FFFFu) >> 4);  // start address, bits [0,14)
    d |= (uint64_t)1 << 16;                               // leading byte offset (unused here), bits [16,30)
    d |= (uint64_t)(1024 >> 4) << 32;                     // stride byte offset, bits [32,46)
    d |= (uint64_t)1 << 46;                               // version, bits [46,48)
    d |= (uint64_t)2 << 61;                               // 128-byte swizzle, bits [61,64)
    return d;
}

// Instruction descriptor: fp32 accumulate, bf16 x bf16, both K-major, N = 128, M = 128.
constexpr uint32_t kTcInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTcN >> 3) << 17) | ((uint32_t)(kTcM >> 4) << 24);

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}" ::"r"(tmem_d),
        "l"(desc_a), "l"(desc_b), "r"(kTcInstrDesc), "r"(accumulate), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t mbar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mbar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

// Thread-block cluster helpers (K split over a cluster, see below, cfi_dense_split.cuh and cfi_slab.cuh).
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_size() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
// Every thread of every CTA of the cluster; writes to shared memory before it are visible to reads through
// distributed shared memory after it.
__device__ __forceinline__ void cluster_sync_all() {
    __syncwarp();
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The same meeting point without ordering any memory: for "every CTA is done reading its peers' shared memory", where
// nothing is published.  (A releasing arrival would first wait for the CTA's outstanding global stores.)
__device__ __forceinline__ void cluster_sync_all_relaxed() {
    __syncwarp();
    asm volatile("barrier.cluster.arrive.relaxed.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
}
// 16 bytes at the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float4 v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "r"(remote)
                 : "memory");
    return v;
}

// Activation for the epilogue, chosen at compile time.  GELU is v * Phi(v) with Phi = (1 + erf(v / sqrt 2)) / 2;
// erf is evaluated with the rational-times-Gaussian formula of Abramowitz & Stegun 7.1.26 (absolute error
// below 1.5e-7, far inside a bf16 result), with the factors 1/sqrt 2 and 1/2 folded into its constants, and
// the two signs of v are kept apart so that the small tail is not obtained by cancellation.
template <int ACT>
__device__ __forceinline__ float activate_tc(float v) {
    if constexpr (ACT != CFI_ACT_GELU_ERF) {
        return v;
    } else {
        float t;  // 1 / (1 + 0.3275911 |v| / sqrt 2)
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(fabsf(v), 0.23164189f, 1.0f)));
        float p = fmaf(0.5307027145f, t, -0.7265760135f);  // half the published coefficients
        p = fmaf(p, t, 0.7107068705f);
        p = fmaf(p, t, -0.142248368f);
        p = fmaf(p, t, 0.127414796f);
        float e;  // exp(-v^2 / 2) = 2^(-v^2 * log2(e) / 2)
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(v * v * -0.72134752f));
        const float m = v * (p * t * e);  // v * (1 - erf(|v| / sqrt 2)) / 2
        return v < 0.0f ? m : v - m;
    }
}

// Two fp32 numbers in one 64-bit register, for the packed fp32 instructions of sm_100 (one issue slot for two
// results: the epilogue of a GELU layer is bound by instruction issue, not by the tensor pipe).
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// act(acc + bias) of two neighbouring outputs, rounded to bf16 and packed (first output in the low half).
// The GELU is the formula of activate_tc with its polynomial and products in packed fp32, and with the two
// signs of v merged into one expression: with q = p t e (a function of |v|, 0 < q <= 1/2),
// v Phi(v) = max(v, 0) - |v| q for either sign, and the negative tail is still a plain product.
template <int ACT>
__device__ __forceinline__ uint32_t bias_act_bf16x2(float a0, float a1, float b0, float b1) {
    float r0, r1;
    if constexpr (ACT != CFI_ACT_GELU_ERF) {
        r0 = a0 + b0;
        r1 = a1 + b1;
    } else {
        float v0, v1, t0, t1, e0, e1, q0, q1;
        const uint64_t v = f2_add(f2_pack(a0, a1), f2_pack(b0, b1));
        f2_unpack(v, v0, v1);
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t0) : "f"(fmaf(fabsf(v0), 0.23164189f, 1.0f)));
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t1) : "f"(fmaf(fabsf(v1), 0.23164189f, 1.0f)));
        const uint64_t t = f2_pack(t0, t1);
        uint64_t p = f2_fma(f2_pack(0.5307027145f, 0.5307027145f), t, f2_pack(-0.7265760135f, -0.7265760135f));
        p = f2_fma(p, t, f2_pack(0.7107068705f, 0.7107068705f));
        p = f2_fma(p, t, f2_pack(-0.142248368f, -0.142248368f));
        p = f2_fma(p, t, f2_pack(0.127414796f, 0.127414796f));
        const uint64_t x2 = f2_mul(f2_mul(v, f2_pack(-0.72134752f, -0.72134752f)), v);  // -v^2 log2(e) / 2
        float s0, s1;
        f2_unpack(x2, s0, s1);
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(s0));
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(s1));
        const uint64_t q = f2_mul(f2_mul(p, t), f2_pack(e0, e1));
        f2_unpack(q, q0, q1);
        r0 = fmaf(-fabsf(v0), q0, fmaxf(v0, 0.0f));
        r1 = fmaf(-fabsf(v1), q1, fmaxf(v1, 0.0f));
    }
    const __nv_bfloat162 pk = __floats2bfloat162_rn(r0, r1);
    return *reinterpret_cast<const uint32_t*>(&pk);
}

// Shared memory (offsets from the first 1024-byte boundary): the ring, then barriers and small tables.
//   ring      kTcStages x [A 128 x 64 bf16 | B 128 x 64 bf16]; after the main loop its first 32 KB hold the y tile
//   +0        full[kTcStages], +32 empty[kTcStages], +64 accumulator barrier, +72 tensor-memory base address
//   +128      bias of the tile's 128 output rows
template <int ACT>
__global__ void __launch_bounds__(kTcThreads, 2)
cfi_dense_tc_kernel(DevLayer L, const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                    __nv_bfloat16* __restrict__ y, int batch) {
    pdl_launch_dependents();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t base = ((smem_u32(0) + 1023u) & ~1023u) - smem_u32(0);  // offset of the first 1024-byte boundary
    const uint32_t ring = base, ctl = base + kTcStages * kTcStageBytes;
    const uint32_t full0 = smem_u32(ctl), empty0 = smem_u32(ctl + 32), accum = smem_u32(ctl + 64);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_at(ctl + 72));
    float* bias_s = reinterpret_cast<float*>(smem_at(ctl + 128));
    const int m0 = blockIdx.y * kTcM, n0 = blockIdx.x * kTcN;
    const int k_blocks_all = (L.in + kTcK - 1) / kTcK;
    // This CTA's share of the K blocks: [kb0, kb0 + k_blocks).
    const int split = (int)cluster_rank(), n_split = (int)cluster_size();
    const int kb0 = (int)(((int64_t)k_blocks_all * split) / n_split);
    const int k_blocks = (int)(((int64_t)k_blocks_all * (split + 1)) / n_split) - kb0;

    if (tid == 0) {
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_w);
        for (int s = 0; s < kTcStages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(accum, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {  // one warp allocates the accumulator's 128 columns of tensor memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(ctl + 72)), "r"(128u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid >= 64 && tid < 64 + kTcN) {
        const int n = n0 + tid - 64;
        bias_s[tid - 64] = n < L.out ? L.bias[n] : 0.0f;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    // The weight belongs to no earlier kernel: its boxes of the first ring round are requested before the wait for
    // the kernel ahead (each slot's barrier already expects the x box too).
    if (warp == 0 && lane == 0) {
        for (int kb = 0; kb < k_blocks && kb < kTcStages; ++kb) {
            mbar_expect_tx(full0 + 8 * kb, kTcStageBytes);
            tma_load_2d(smem_u32(ring + kb * kTcStageBytes) + kTcM * kTcK * 2, &map_w, full0 + 8 * kb, (kb0 + kb) * kTcK, n0);
        }
    }
    pdl_wait();  // x and y may belong to the kernel before this one
    bool ok = true;
    int issued = 0;  // thread 0: K blocks whose boxes it has requested

    if (warp == 0 && lane == 0) {
        // ---------------------------------------------------------------- TMA producer
        for (int kb = 0; kb < k_blocks && ok; ++kb) {
            const int s = kb % kTcStages;
            if (kb >= kTcStages) ok = mbar_wait(empty0 + 8 * s, (uint32_t)(kb / kTcStages - 1) & 1u, kTcSpinLimit);
            if (!ok) break;
            const uint32_t a_dst = smem_u32(ring + s * kTcStageBytes), b_dst = a_dst + kTcM * kTcK * 2;
            if (kb >= kTcStages) mbar_expect_tx(full0 + 8 * s, kTcStageBytes);
            tma_load_2d(a_dst, &map_x, full0 + 8 * s, (kb0 + kb) * kTcK, m0);
            if (kb >= kTcStages) tma_load_2d(b_dst, &map_w, full0 + 8 * s, (kb0 + kb) * kTcK, n0);
            issued = kb + 1;  // (the first ring round has no wait that could fail, so no stage is left with only its weight box)
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------------------------------------------------------- MMA issuer
        for (int kb = 0; kb < k_blocks && ok; ++kb) {
            const int s = kb % kTcStages;
            ok = mbar_wait(full0 + 8 * s, (uint32_t)(kb / kTcStages) & 1u, kTcSpinLimit);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_addr = smem_u32(ring + s * kTcStageBytes), b_addr = a_addr + kTcM * kTcK * 2;
            const uint64_t da = umma_desc_k_sw128(a_addr), db = umma_desc_k_sw128(b_addr);
#pragma unroll
            for (int k = 0; k < kTcK / 16; ++k)  // 16 bf16 = 32 bytes further along K inside the swizzled row
                umma_bf16(tmem_base, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), (kb | k) != 0 ? 1u : 0u);
            umma_commit(empty0 + 8 * s);  // the slot is free once these MMAs have read it
        }
        umma_commit(accum);  // the accumulator is complete once every MMA issued so far has finished (also after a failed wait)
    } else if (warp >= 2) {
        // ---------------------------------------------------------------- epilogue
        ok = mbar_wait(accum, 0u, kTcSpinLimit);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int q = warp & 3;            // a warp may read the tensor-memory lanes 32 q .. 32 q + 31
        const int half = (warp - 2) >> 2;  // two warps share a lane quarter and split the 128 columns
        const int row = 32 * q + lane;     // batch row of the tile held by this thread
        if (ok && n_split > 1) {
            // Partial tile, fp32, no bias: 128 rows x 512 bytes, 16-byte chunks permuted by chunk ^ (row & 15).
#pragma unroll 1
            for (int c = 64 * half; c < 64 * half + 64; c += 16) {
                uint32_t v[16];
                tmem_ld16(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)c, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int e4 = 0; e4 < 4; ++e4) {
                    float4 r = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                    if (k_blocks > 0)  // a CTA without K blocks has issued no MMA: its accumulator holds nothing
                        r = make_float4(__uint_as_float(v[4 * e4]), __uint_as_float(v[4 * e4 + 1]), __uint_as_float(v[4 * e4 + 2]),
                                        __uint_as_float(v[4 * e4 + 3]));
                    const int ch = (c >> 2) + e4;
                    *reinterpret_cast<float4*>(smem_at(ring + row * 512 + ((ch ^ (row & 15)) << 4))) = r;
                }
            }
        } else if (ok) {
            // y tile in shared memory: 128 rows x 256 bytes, 16-byte chunks permuted by chunk ^ (row & 15).
#pragma unroll 1
            for (int c = 64 * half; c < 64 * half + 64; c += 32) {
                uint32_t v[2][16];
                tmem_ld16(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)c, v[0]);
                tmem_ld16(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(c + 16), v[1]);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t packed[8];
#pragma unroll
                    for (int e4 = 0; e4 < 4; ++e4) {
                        const float4 bv = *reinterpret_cast<const float4*>(bias_s + c + 16 * h + 4 * e4);
                        packed[2 * e4] = bias_act_bf16x2<ACT>(__uint_as_float(v[h][4 * e4 + 0]), __uint_as_float(v[h][4 * e4 + 1]), bv.x, bv.y);
                        packed[2 * e4 + 1] = bias_act_bf16x2<ACT>(__uint_as_float(v[h][4 * e4 + 2]), __uint_as_float(v[h][4 * e4 + 3]), bv.z, bv.w);
                    }
                    const int ch = (c + 16 * h) >> 3;  // 16-byte chunk of columns .. +7; the next one holds +8 .. +15
                    *reinterpret_cast<uint4*>(smem_at(ring + row * 256 + ((ch ^ (row & 15)) << 4))) =
                        make_uint4(packed[0], packed[1], packed[2], packed[3]);
                    *reinterpret_cast<uint4*>(smem_at(ring + row * 256 + (((ch + 1) ^ (row & 15)) << 4))) =
                        make_uint4(packed[4], packed[5], packed[6], packed[7]);
                }
            }
        }
        if (n_split == 1) asm volatile("bar.sync 1, %0;" ::"n"(32 * kTcEpilogueWarps) : "memory");  // the epilogue warps only
        if (ok && n_split == 1) {
            const int et = tid - 64;  // 16 threads per row, 16 rows per pass
            for (int r = et >> 4; r < kTcM; r += 2 * kTcEpilogueWarps) {
                const int ch = et & 15, m = m0 + r, n = n0 + 8 * ch;
                if (m < batch && n < L.out) {
                    const uint4 val = *reinterpret_cast<const uint4*>(smem_at(ring + r * 256 + ((ch ^ (r & 15)) << 4)));
                    *reinterpret_cast<uint4*>(y + (size_t)m * L.out + n) = val;
                }
            }
        }
    }
    if (n_split > 1) {
        // Every thread of every CTA of the cluster passes both barriers, whatever `ok` says.
        cluster_sync_all();  // the partial tiles are complete
        if (warp >= 2 && ok) {
            // Rows [split * rows_per, (split + 1) * rows_per): sum over the cluster in rank order, bias, activation,
            // bf16, store.  32 threads per row (4 columns each), 8 rows per pass, 256-byte runs.
            const int et = tid - 64, ch = et & 31, rows_per = (kTcM + n_split - 1) / n_split, n = n0 + 4 * ch;
            const float4 bv = *reinterpret_cast<const float4*>(bias_s + 4 * ch);
            for (int rr = et >> 5; rr < rows_per; rr += kTcEpilogueWarps) {
                const int r = split * rows_per + rr, m = m0 + r;
                if (r < kTcM && m < batch && n < L.out) {
                    const uint32_t off = smem_u32(ring + r * 512 + ((ch ^ (r & 15)) << 4));
                    float4 a = ld_cluster_f4(off, 0u);
                    for (int p = 1; p < n_split; ++p) {
                        const float4 t = ld_cluster_f4(off, (uint32_t)p);
                        a.x += t.x, a.y += t.y, a.z += t.z, a.w += t.w;
                    }
                    const __nv_bfloat162 p01 = __floats2bfloat162_rn(activate_tc<ACT>(a.x + bv.x), activate_tc<ACT>(a.y + bv.y));
                    const __nv_bfloat162 p23 = __floats2bfloat162_rn(activate_tc<ACT>(a.z + bv.z), activate_tc<ACT>(a.w + bv.w));
                    *reinterpret_cast<uint2*>(y + (size_t)m * L.out + n) =
                        make_uint2(*reinterpret_cast<const uint32_t*>(&p01), *reinterpret_cast<const uint32_t*>(&p23));
                }
            }
        }
        cluster_sync_all_relaxed();  // no CTA leaves while another may still read its tile
    }
    if (!ok) atomicExch(L.status, 2);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    if (__syncthreads_or(!ok)) {
        // A wait gave up somewhere in this CTA.  It must not end while a box is still on its way into its shared memory
        // (the copy would land in, and signal a barrier of, whichever CTA gets that memory next) or while an MMA still
        // works on its tensor memory: wait, again bounded, for the boxes requested and for the issuer's last commit.
        if (tid == 0) {
            for (int j = issued > kTcStages ? issued - kTcStages : 0; j < issued; ++j)
                mbar_wait(full0 + 8 * (j % kTcStages), (uint32_t)(j / kTcStages) & 1u, kTcSpinLimit);
            mbar_wait(accum, 0u, kTcSpinLimit);
        }
        __syncthreads();
    }
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(128u) : "memory");
    }
}
