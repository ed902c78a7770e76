// CFI_VARIANT_DENSE_TC for fp32 layers: the dense contraction on the tensor cores in split TF32.
//
// Included by cfi_layer.cu after cfi_dense_tc.cuh (it reuses that file's mbarrier, TMA, descriptor and
// tensor-memory helpers).
//
// A TF32 operand keeps 11 significant bits of an fp32 number, which alone would miss the 1e-5 tolerance of
// the fp32 layer by two orders of magnitude.  Each operand is therefore split into two TF32-exact parts,
//
//     a = a_hi + a_lo + r,   a_hi = a with the low 13 mantissa bits cleared,   a_lo = (a - a_hi) likewise cleared,
//
// so that |r| < 2^-21 |a|, and the product is taken as  x_hi w_hi + x_hi w_lo + x_lo w_hi  (three products in
// two MMAs, fp32 accumulation in tensor memory).  What is dropped (x_lo w_lo and the two remainders) is below 2^-19 of the
// term, fifty times inside the tolerance.  Because both parts are exactly representable in TF32, the result
// does not depend on how the tensor core would convert a general fp32 operand.
//
// The layer keeps one dense fp32 copy of its weight, Wd[out_pad][in].  Per 32-column block of K:
//   warp 0, one lane   TMA: a 128 x 32 box of x and a TN x 32 box of Wd (fp32, 128-byte swizzle) into a ring slot;
//   warps 2..17        four groups of four warps; group g takes the blocks kb = g (mod 4), so four blocks are being
//                      split at once.  A thread reads its batch row of the x box from shared memory and writes
//                      hi and lo straight into tensor memory (tcgen05.st), from where the MMA takes its A
//                      operand, so x costs shared-memory bandwidth once instead of once per MMA; the group also
//                      splits the Wd box in shared memory, hi in place and lo beside it (element-wise, so the
//                      swizzled layout is untouched), and makes those writes visible to the tensor core
//                      (fence.proxy.async);
//   warp 1, one lane   once the group's 128 threads have arrived on the slot's "ready" barrier: 4 K-steps x 2
//                      tcgen05.mma (kind::tf32, M = 128, K = 8, A from tensor memory, B from shared memory): Wd lo
//                      lies right behind Wd hi, so x_hi x [Wd hi; Wd lo] is one MMA of N = 2 TN (the two products
//                      land in accumulator columns 0..TN-1 and TN..2TN-1) and x_lo x Wd hi a second of N = TN onto
//                      the first half; then tcgen05.commit frees the slot.  (An MMA costs about 50 cycles + 0.43 per
//                      column of N here, so fewer and wider MMAs win; hence also the tile width TN = 128 where the
//                      shape gives enough tiles.)
// and after the last block warps 2..17 run the epilogue: tcgen05.ld of both accumulator halves, their sum, bias,
// activation, y tile through shared memory, runs of 4 TN bytes per batch row.  Tensor memory: 2 TN accumulator
// columns, then per slot 32 columns of x_hi and 32 of x_lo.  All mbarrier waits are bounded (status code 2), as in
// the bf16 kernel.
//
// Split K over a thread-block cluster: a layer with few output tiles and a long K (3072 -> 768 at batch 256 has 24
// tiles of 96 K blocks) would leave most SMs idle, so the launch may give each tile to a cluster of up to 8 CTAs
// (cluster dimension z).  CTA r of the cluster contracts the r-th share of the K blocks; the partial tiles are left
// in each CTA's shared memory, and after a cluster barrier CTA r sums rows [128 r / S, 128 (r + 1) / S) of all S
// partial tiles in rank order through distributed shared memory, adds the bias, applies the activation and stores
// them.  The barrier is the hardware cluster barrier (no flags, no global workspace), the order of additions is
// fixed, and the layer stays read-only, so concurrent calls on one layer remain safe.

constexpr int kTfM = 128, kTfK = 32, kTfStages = 4;  // the output tile is kTfM x TN with TN = 64, 96 or 128 (template)
constexpr int kTfGroups = 4;  // groups of four worker warps; group g splits the K blocks kb with kb % kTfGroups == g
constexpr int kTfWorkerWarps = 4 * kTfGroups, kTfThreads = 64 + 32 * kTfWorkerWarps;
// A ring slot is always split by the same group, so that one phase bit per barrier is enough: a group that ran a
// whole phase ahead on another group's slot would pass its wait early.
static_assert(kTfStages == kTfGroups, "slot s belongs to group s");
constexpr uint32_t kTfABytes = kTfM * kTfK * 4;                                 // x box: 16 KB
constexpr uint32_t kTfTmemCols = 512;  // 2 TN accumulator columns (x_hi w_hi + x_lo w_hi | x_hi w_lo) + 4 slots of 64
__host__ __device__ constexpr uint32_t tf_b_bytes(int tn) { return (uint32_t)tn * kTfK * 4; }  // Wd box: 8 or 16 KB
__host__ __device__ constexpr uint32_t tf_stage_bytes(int tn) { return kTfABytes + 2 * tf_b_bytes(tn); }  // x | Wd hi | Wd lo
__host__ __device__ constexpr size_t tf_smem_bytes(int tn) { return 1024 + (size_t)kTfStages * tf_stage_bytes(tn) + 1024; }

// fp32 accumulate, tf32 x tf32, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t tf_instr_desc(int n) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTfM >> 4) << 24);
}

// A operand from tensor memory (row m in lane m, 32-bit elements in consecutive columns), B from shared memory.
__device__ __forceinline__ void umma_tf32_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}" ::"r"(tmem_d),
        "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t mbar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(mbar) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(
            taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

// Sum of the 16 bytes at shared-memory address `addr` over the S CTAs of the cluster, in rank order, for each of
// ITER rows that are `row_step` bytes apart.  All S * ITER loads are issued before the first sum needs one, so the
// latency of distributed shared memory is paid once, and the CTA's own tile is read as ordinary shared memory.
template <int S, int ITER>
__device__ __forceinline__ void cluster_sum_rows(uint32_t addr, uint32_t row_step, uint32_t own_rank, float4 (&out)[ITER]) {
    float4 t[ITER][S];
#pragma unroll
    for (int it = 0; it < ITER; ++it)
#pragma unroll
        for (int p = 0; p < S; ++p) {
            const uint32_t a = addr + (uint32_t)it * row_step;
            if ((uint32_t)p == own_rank) {
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                             : "=f"(t[it][p].x), "=f"(t[it][p].y), "=f"(t[it][p].z), "=f"(t[it][p].w)
                             : "r"(a)
                             : "memory");
            } else {
                t[it][p] = ld_cluster_f4(a, (uint32_t)p);
            }
        }
#pragma unroll
    for (int it = 0; it < ITER; ++it) {
        out[it] = t[it][0];
#pragma unroll
        for (int p = 1; p < S; ++p) out[it].x += t[it][p].x, out[it].y += t[it][p].y, out[it].z += t[it][p].z, out[it].w += t[it][p].w;
    }
}

// hi = v with the 13 low mantissa bits cleared; lo = the same of (v - hi).  Both are exact TF32 numbers.
__device__ __forceinline__ void split_tf32(float v, float& hi, float& lo) {
    hi = __uint_as_float(__float_as_uint(v) & 0xFFFFE000u);
    lo = __uint_as_float(__float_as_uint(v - hi) & 0xFFFFE000u);
}

// Shared memory from the first 1024-byte boundary: kTfStages slots of [x raw | Wd hi | Wd lo]; then
//   +0 full[4], +32 ready[4], +64 empty[4], +96 accumulator barrier, +104 tensor-memory base, +128 bias[TN].
template <int TN>
__global__ void __launch_bounds__(kTfThreads, 1)
cfi_dense_tf32_kernel(DevLayer L, const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                      float* __restrict__ y, int batch) {
    pdl_launch_dependents();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t base = ((smem_u32(0) + 1023u) & ~1023u) - smem_u32(0);
    static_assert(TN == 64 || TN == 96 || TN == 128, "tile width");
    // Partial tile in shared memory: 16-byte chunk c of row r sits at c ^ (r & kPermMask); the mask keeps the chunk
    // inside its aligned group of 16 (or of 8 where a row has 24 chunks).
    constexpr uint32_t kPermMask = TN % 64 == 0 ? 15u : 7u;
    constexpr uint32_t kBBytes = tf_b_bytes(TN), kStageBytes = tf_stage_bytes(TN), kAccCols = 2 * TN;
    static_assert(kAccCols + 64 * kTfStages <= kTfTmemCols, "tensor memory: accumulators + x slots");
    const uint32_t ring = base, ctl = base + kTfStages * kStageBytes;
    const uint32_t full0 = smem_u32(ctl), ready0 = smem_u32(ctl + 32), empty0 = smem_u32(ctl + 64), accum = smem_u32(ctl + 96);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_at(ctl + 104));
    float* bias_s = reinterpret_cast<float*>(smem_at(ctl + 128));
    const int m0 = blockIdx.y * kTfM, n0 = blockIdx.x * TN;
    const int k_blocks = (L.in + kTfK - 1) / kTfK;
    // This CTA's share of the K blocks: [kb0, kb0 + n_local).
    const int split = (int)cluster_rank(), n_split = (int)cluster_size();
    const int kb0 = (int)(((int64_t)k_blocks * split) / n_split);
    const int n_local = (int)(((int64_t)k_blocks * (split + 1)) / n_split) - kb0;

    if (tid == 0) {
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_w);
        for (int s = 0; s < kTfStages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(ready0 + 8 * s, 128);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(accum, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(ctl + 104)), "r"(kTfTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // The bias is read only after the main loop (and after a barrier), so its load from global memory is issued
    // here and lands in shared memory after the prologue's barrier instead of holding it up.
    float bias_v = 0.0f;
    if (tid >= 64 && tid < 64 + TN && n0 + tid - 64 < L.out) bias_v = L.bias[n0 + tid - 64];
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    // The layer's weight belongs to no earlier kernel: the Wd boxes of the first ring round are requested before
    // the wait for the kernel ahead (their slots' barriers already expect the x box as well), so a cold weight
    // streams in while that kernel finishes.
    if (warp == 0 && lane == 0) {
        for (int i = 0; i < n_local && i < kTfStages; ++i) {
            mbar_expect_tx(full0 + 8 * i, kTfABytes + kBBytes);
            tma_load_2d(smem_u32(ring + i * kStageBytes) + kTfABytes, &map_w, full0 + 8 * i, (kb0 + i) * kTfK, n0);
        }
    }
    pdl_wait();  // x and y may belong to the kernel before this one
    if (tid >= 64 && tid < 64 + TN) bias_s[tid - 64] = bias_v;
    bool ok = true;

    if (warp == 0 && lane == 0) {
        // ---------------------------------------------------------------- TMA producer
        for (int i = 0; i < n_local && ok; ++i) {
            const int s = i % kTfStages;
            if (i >= kTfStages) ok = mbar_wait(empty0 + 8 * s, (uint32_t)(i / kTfStages - 1) & 1u, kTcSpinLimit);
            if (!ok) break;
            const uint32_t a_dst = smem_u32(ring + s * kStageBytes), b_dst = a_dst + kTfABytes;
            if (i >= kTfStages) mbar_expect_tx(full0 + 8 * s, kTfABytes + kBBytes);
            tma_load_2d(a_dst, &map_x, full0 + 8 * s, (kb0 + i) * kTfK, m0);
            if (i >= kTfStages) tma_load_2d(b_dst, &map_w, full0 + 8 * s, (kb0 + i) * kTfK, n0);
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------------------------------------------------------- MMA issuer
        for (int i = 0; i < n_local && ok; ++i) {
            const int s = i % kTfStages;
            ok = mbar_wait(ready0 + 8 * s, (uint32_t)(i / kTfStages) & 1u, kTcSpinLimit);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t b_hi = smem_u32(ring + s * kStageBytes + kTfABytes);  // Wd lo follows at + kBBytes
            const uint64_t dbh = umma_desc_k_sw128(b_hi);
            const uint32_t a_hi = tmem_base + kAccCols + (uint32_t)(64 * s), a_lo = a_hi + 32u;
#pragma unroll
            for (int k = 0; k < kTfK / 8; ++k) {  // 8 fp32 further along K: 8 columns of tensor memory, 32 bytes of a row
                const uint64_t off = (uint64_t)(2 * k);
                // Wd lo lies right behind Wd hi, so the two boxes read as one K-major operand of 2 TN rows: one MMA
                // of N = 2 TN gives x_hi w_hi in columns 0..TN-1 and x_hi w_lo in columns TN..2TN-1; a second of
                // N = TN adds x_lo w_hi to the first half.  (An MMA costs about 50 cycles + 0.43 per column of N.)
                umma_tf32_ts(tmem_base, a_hi + 8u * k, dbh + off, tf_instr_desc(2 * TN), (i | k) != 0 ? 1u : 0u);
                umma_tf32_ts(tmem_base, a_lo + 8u * k, dbh + off, tf_instr_desc(TN), 1u);
            }
            umma_commit(empty0 + 8 * s);
        }
        if (ok) umma_commit(accum);
    } else if (warp >= 2) {
        // ---------------------------------------------------------------- split, then epilogue
        const int wt = tid - 64;            // 0 .. 32 * kTfWorkerWarps - 1
        const int group = (warp - 2) >> 2;  // the group's four warps cover the four lane quarters of tensor memory
        const int gt = wt & 127;            // thread within the group
        for (int i = group; i < n_local && ok; i += kTfGroups) {
            const int s = i % kTfStages;
            ok = mbar_wait(full0 + 8 * s, (uint32_t)(i / kTfStages) & 1u, kTcSpinLimit);
            if (!ok) break;
            {
                // x: this thread's batch row (tensor-memory lane): 8 chunks of 16 bytes, un-permuted from the
                // swizzle, split and written straight to tensor memory.
                const int m = 32 * (warp & 3) + lane;
                const uint32_t row_off = ring + s * kStageBytes + (uint32_t)m * 128u;
                const uint32_t t_hi = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + kAccCols + (uint32_t)(64 * s);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t hi[16], lo[16];
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const float4 v =
                            *reinterpret_cast<const float4*>(smem_at(row_off + (uint32_t)(((4 * half + c) ^ (m & 7)) << 4)));
                        float h, l;
                        split_tf32(v.x, h, l), hi[4 * c + 0] = __float_as_uint(h), lo[4 * c + 0] = __float_as_uint(l);
                        split_tf32(v.y, h, l), hi[4 * c + 1] = __float_as_uint(h), lo[4 * c + 1] = __float_as_uint(l);
                        split_tf32(v.z, h, l), hi[4 * c + 2] = __float_as_uint(h), lo[4 * c + 2] = __float_as_uint(l);
                        split_tf32(v.w, h, l), hi[4 * c + 3] = __float_as_uint(h), lo[4 * c + 3] = __float_as_uint(l);
                    }
                    tmem_st16(t_hi + 16u * half, hi);
                    tmem_st16(t_hi + 32u + 16u * half, lo);
                }
                // Wd: element-wise, hi in place, lo beside it (TN / 16 of its 8 TN 16-byte pieces per thread).
                const uint32_t hi_off = ring + s * kStageBytes + kTfABytes, lo_off = hi_off + kBBytes;
#pragma unroll
                for (uint32_t e = (uint32_t)gt * 16u; e < kBBytes; e += 128u * 16u) {
                    const float4 v = *reinterpret_cast<const float4*>(smem_at(hi_off + e));
                    float4 h, l;
                    split_tf32(v.x, h.x, l.x);
                    split_tf32(v.y, h.y, l.y);
                    split_tf32(v.z, h.z, l.z);
                    split_tf32(v.w, h.w, l.w);
                    *reinterpret_cast<float4*>(smem_at(hi_off + e)) = h;
                    *reinterpret_cast<float4*>(smem_at(lo_off + e)) = l;
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> visible to the MMA's reads
            mbar_arrive(ready0 + 8 * s);
        }
        ok = __all_sync(0xffffffffu, ok);
        if (ok) ok = mbar_wait(accum, 0u, kTcSpinLimit);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int q = warp & 3;  // tensor-memory lanes 32 q .. 32 q + 31; the group number picks TN / 4 of the TN columns
        const int row = 32 * q + lane;
        if (ok) {
            // This CTA's partial tile (no bias yet) in shared memory: 128 rows of 4 TN bytes, 16-byte chunks permuted
            // by chunk ^ (row & 15).  The two accumulator halves are the two groups of products.
#pragma unroll
            for (int ck = 0; ck < (TN / 16 + kTfGroups - 1) / kTfGroups; ++ck) {
                const int col0 = 16 * (group + kTfGroups * ck);  // the groups take the 16-column pieces in turn
                if (col0 >= TN) break;                           // (the same for a whole warp)
                uint32_t v[16], v1[16];
                const uint32_t t_acc = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)col0;
                tmem_ld16(t_acc, v);
                tmem_ld16(t_acc + TN, v1);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int e4 = 0; e4 < 4; ++e4) {
                    const int col = col0 + 4 * e4;
                    float4 r = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                    if (n_local > 0) {  // a CTA without K blocks has issued no MMA: its accumulator holds nothing
                        r.x = __uint_as_float(v[4 * e4 + 0]) + __uint_as_float(v1[4 * e4 + 0]);
                        r.y = __uint_as_float(v[4 * e4 + 1]) + __uint_as_float(v1[4 * e4 + 1]);
                        r.z = __uint_as_float(v[4 * e4 + 2]) + __uint_as_float(v1[4 * e4 + 2]);
                        r.w = __uint_as_float(v[4 * e4 + 3]) + __uint_as_float(v1[4 * e4 + 3]);
                    }
                    *reinterpret_cast<float4*>(smem_at(ring + row * (4 * TN) + (((col >> 2) ^ (row & kPermMask)) << 4))) = r;
                }
            }
        }
        if (n_split == 1) asm volatile("bar.sync 1, %0;" ::"n"(32 * kTfWorkerWarps) : "memory");
    }
    // The partial tiles of the whole cluster are complete: every thread of every CTA passes here, whatever `ok` says.
    if (n_split > 1) cluster_sync_all();
    if (warp >= 2 && ok) {
        // Rows [split * rows_per, (split + 1) * rows_per) of the tile: sum over the cluster in rank order, bias,
        // activation, store.  TN / 4 threads per row, runs of 4 TN bytes.
        // (24 threads per row do not divide the 512 workers: at TN = 96 the first 384 take 16 rows per pass.)
        constexpr int kPerRow = TN / 4, kRowsPerPass = TN == 96 ? 16 : 32 * kTfWorkerWarps / kPerRow;
        const int wt = tid - 64, ch = wt % kPerRow, rows_per = (kTfM + n_split - 1) / n_split;
        const float4 bv = *reinterpret_cast<const float4*>(bias_s + 4 * ch);
        const int n = n0 + 4 * ch;
        // Clusters of 2, 4 and 8: the thread's rows are kRowsPerPass apart (a multiple of 16, so the chunk
        // permutation is the same for all of them) and all their loads are issued together.
        auto fast = [&](auto s_tag, auto iter_tag) {
            constexpr int S = decltype(s_tag)::value, ITER = decltype(iter_tag)::value;
            const int rr0 = wt / kPerRow;
            if (rr0 >= kTfM / S || rr0 >= kRowsPerPass) return;
            const int r0 = split * (kTfM / S) + rr0;
            float4 acc[ITER];
            cluster_sum_rows<S, ITER>(smem_u32(ring + r0 * (4 * TN) + ((ch ^ (r0 & kPermMask)) << 4)), kRowsPerPass * 4 * TN,
                                      (uint32_t)split, acc);
#pragma unroll
            for (int it = 0; it < ITER; ++it) {
                const int m = m0 + r0 + it * kRowsPerPass;
                if (m < batch && n < L.out) {
                    float4 a = acc[it];
                    a.x = activate(a.x + bv.x, L.act);
                    a.y = activate(a.y + bv.y, L.act);
                    a.z = activate(a.z + bv.z, L.act);
                    a.w = activate(a.w + bv.w, L.act);
                    *reinterpret_cast<float4*>(y + (size_t)m * L.out + n) = a;
                }
            }
        };
        using std::integral_constant;
        constexpr int kIter2 = kTfM / 2 / kRowsPerPass, kIter4 = kTfM / 4 / kRowsPerPass;
        if (n_split == 2) fast(integral_constant<int, 2>{}, integral_constant<int, kIter2>{});
        else if (n_split == 4) fast(integral_constant<int, 4>{}, integral_constant<int, (kIter4 > 0 ? kIter4 : 1)>{});
        else if (n_split == 8) fast(integral_constant<int, 8>{}, integral_constant<int, 1>{});
        else if (wt < kRowsPerPass * kPerRow)
        for (int rr = wt / kPerRow; rr < rows_per; rr += kRowsPerPass) {
            const int r = split * rows_per + rr, m = m0 + r;
            if (r < kTfM && m < batch && n < L.out) {
                const uint32_t off = ring + r * (4 * TN) + ((ch ^ (r & kPermMask)) << 4);
                float4 a;
                if (n_split == 1) {
                    a = *reinterpret_cast<const float4*>(smem_at(off));
                } else {
                    a = ld_cluster_f4(smem_u32(off), 0u);
                    for (int p = 1; p < n_split; ++p) {
                        const float4 t = ld_cluster_f4(smem_u32(off), (uint32_t)p);
                        a.x += t.x, a.y += t.y, a.z += t.z, a.w += t.w;
                    }
                }
                a.x = activate(a.x + bv.x, L.act);
                a.y = activate(a.y + bv.y, L.act);
                a.z = activate(a.z + bv.z, L.act);
                a.w = activate(a.w + bv.w, L.act);
                *reinterpret_cast<float4*>(y + (size_t)m * L.out + n) = a;
            }
        }
    }
    if (n_split > 1) cluster_sync_all_relaxed();  // no CTA leaves while another may still read its tile
    if (!ok) atomicExch(L.status, 2);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTfTmemCols) : "memory");
    }
}
