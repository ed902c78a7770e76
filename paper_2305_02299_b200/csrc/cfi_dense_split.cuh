// CFI_VARIANT_DENSE_TC for fp32 layers: the dense contraction on the tensor cores in split TF32, with the weight as
// the M operand and the batch as the N operand.
//
// Included by cfi_layer.cu after cfi_dense_tc.cuh (it reuses that file's mbarrier, TMA, descriptor, tensor-memory and
// cluster helpers).
//
// A TF32 operand keeps 11 significant bits of an fp32 number, which alone would miss the 1e-5 tolerance of the fp32
// layer by two orders of magnitude.  Each operand is therefore split into two TF32-exact parts,
//
//     a = a_hi + a_lo + r,   a_hi = a with the low 13 mantissa bits cleared,   a_lo = (a - a_hi) likewise cleared,
//
// so that |a_lo| < 2^-10 |a| and |r| < 2^-20 |a|, and a product is taken as  w_hi x_hi + w_hi x_lo + w_lo x_hi  (fp32
// accumulation in tensor memory).  What is dropped (w_lo x_lo and the two remainders) is below 3 * 2^-20 of the term
// whatever the signs, three times inside the tolerance even for a fan-in of one.  Both parts are exactly representable
// in TF32, so the result does not depend on how the tensor core would convert a general fp32 operand, and they keep
// fp32's exponent range.  (Two bf16 pieces per operand would halve the bytes and the instructions, but 16 significant
// bits leave up to 3e-5 of a term: not enough.)
//
// The tensor core reads only the upper 19 bits of a TF32 operand (results are bit-identical whether the low 13 bits
// are cleared or not; a part that rounded instead would fail the parity tests at small fan-in by 1e-3), so the hi
// parts are the raw fp32 numbers themselves and only the lo parts have to be computed.
//
// The layer keeps one dense fp32 copy of its weight, Wd[out_pad][in] (zero rows for ablated and padding rows).  A tile
// is 128 output rows (M) x BT batch rows (N side), so a small batch costs a narrow MMA and not a mostly empty 128-row
// tile.  Per 32-column block of K, in a ring of four to eight stages [Wd box | x box | x_lo]:
//   warp 0, one lane    TMA: the 128 x 32 box of Wd and the BT x 32 box of x (fp32, 128-byte swizzle).  The weight
//                       boxes of the first ring round are requested before the wait for the kernel ahead;
//   warps 3..18         two teams of eight worker warps; team t prepares the blocks i = t (mod 2).  x_lo: the x box is
//                       read back from shared memory, x - (x with the low 13 bits cleared) is written right behind
//                       it in the same swizzled layout, so that [x; x_lo] reads as one K-major operand of 2 BT rows.
//                       w_lo: two threads per output row read that row's 128 bytes of the Wd box and write the lo
//                       parts straight into tensor memory (tcgen05.st), from where the second MMA takes its A
//                       operand.  tcgen05.wait::st and fence.proxy.async, then one arrival per warp on the stage's
//                       "ready" barrier;
//   warps 1 and 2, one lane each   two MMA issuers (kind::tf32, M = 128, K = 8).  Warp 1 issues  Wd x [x; x_lo]
//                       (A = the Wd box in shared memory, N = 2 BT) into accumulator columns 0 .. 2BT-1, warp 2 issues
//                       w_lo x x  (A from tensor memory, N = BT) into columns 2BT .. 3BT-1.  One thread gets an MMA
//                       accepted about every 143 cycles whatever its size (measured on this part), two threads get
//                       two; separate accumulators keep the two streams independent.  Each issuer's tcgen05.commit
//                       arrives on the stage's "empty" barrier (count 2), which the TMA lane waits for.
// After the last block the workers add the three accumulator parts, add the bias, apply the activation and store: a
// tensor-memory lane is an output row, so for one batch row a warp writes 32 consecutive outputs, 128 contiguous bytes.
//
// Split K over a thread-block cluster (cluster dimension z) as in the bf16 kernel: CTA r contracts the r-th share of
// the K blocks, leaves its partial tile [BT][128] in its shared memory, and after the hardware cluster barrier sums its
// share of the batch rows over all CTAs in rank order through distributed shared memory.  No flags, no workspace, a
// fixed order of additions, and the layer stays read-only.
// Every mbarrier wait is bounded (status code 2).  After a wait that gave up the CTA still waits, bounded again, for the
// boxes it has requested and for the MMAs it has issued before it frees its tensor memory and ends.

constexpr int kSpM = 128, kSpK = 32;
constexpr int kSpTeamWarps = 8, kSpTeams = 2, kSpWorkerWarps = kSpTeams * kSpTeamWarps, kSpFirstWorker = 3;
constexpr int kSpThreads = 32 * (kSpFirstWorker + kSpWorkerWarps);
// Batch tiles of the kernel (the MMA's N is BT and 2 BT, multiples of 16 up to 256) and the ring depth each one affords
// in shared memory (16 KB + 256 BT bytes per stage) and tensor memory (3 BT accumulator columns + 32 per stage).
constexpr int kSpTiles[] = {16, 32, 48, 64, 96, 128};
constexpr int kSpNumTiles = sizeof(kSpTiles) / sizeof(kSpTiles[0]);
// The depth is a multiple of the number of worker teams, so that a ring slot always belongs to the same team: a team
// that met only every other phase of a slot's barrier could not tell a phase from the one two before it by parity.
__host__ __device__ constexpr int sp_stages(int bt) { return bt >= 96 ? 4 : bt >= 48 ? 6 : 8; }
constexpr int kMaxClusterSplit = 8;  // largest portable thread-block cluster
constexpr uint32_t kSpWBytes = kSpM * kSpK * 4;  // one weight box: 16 KB
constexpr uint32_t kSpTmemCols = 512;            // 3 BT accumulator columns ... one 32-column w_lo stage per ring slot at the top
__host__ __device__ constexpr uint32_t sp_x_bytes(int bt) { return (uint32_t)bt * kSpK * 4; }  // the x box; x_lo has the same size
__host__ __device__ constexpr uint32_t sp_stage_bytes(int bt) { return kSpWBytes + 2 * sp_x_bytes(bt); }
__host__ __device__ constexpr uint32_t sp_data_bytes(int bt) {  // the ring, or the partial tile of a K split if that is larger
    return sp_stages(bt) * sp_stage_bytes(bt) > (uint32_t)bt * 512u ? sp_stages(bt) * sp_stage_bytes(bt) : (uint32_t)bt * 512u;
}
__host__ __device__ constexpr size_t sp_smem_bytes(int bt) { return 1024 + (size_t)sp_data_bytes(bt) + 1024; }

// fp32 accumulate, tf32 x tf32, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t sp_instr_desc(int n) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kSpM >> 4) << 24);
}
// Both operands from shared memory.
__device__ __forceinline__ void umma_tf32_ss(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}" ::"r"(tmem_d),
        "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
// A operand from tensor memory (row m in lane m, 32-bit elements in consecutive columns), B from shared memory.
__device__ __forceinline__ void umma_tf32_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}" ::"r"(tmem_d),
        "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(
            taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
// What the hi part (v itself, of which the tensor core reads the upper 19 bits) leaves over: exact in fp32.
__device__ __forceinline__ float tf32_lo(float v) { return v - __uint_as_float(__float_as_uint(v) & 0xFFFFE000u); }

// The cluster reduction of a K split, for a cluster of NS CTAs: batch rows [split * rows_per, (split + 1) * rows_per)
// of the tile are summed over the CTAs' partial tiles in rank order, then bias, activation, store.  32 threads per
// batch row (4 outputs each), 16 rows per pass, 512-byte runs of y.  The loads of kRows rows (NS each; the CTA's own tile
// is read as ordinary shared memory) are all issued before the first sum needs one, so that the latency of distributed
// shared memory is paid once per kRows rows.
template <int BT, int NS>
__device__ __forceinline__ void sp_reduce(const DevLayer& L, float* __restrict__ y, int batch, int n0, int b0, uint32_t base, int split,
                                          int wt) {
    constexpr int kRows = NS <= 2 ? 4 : NS <= 4 ? 2 : 1;
    const int ch = wt & 31, rows_per = (BT + NS - 1) / NS, o = n0 + 4 * ch;
    if (o >= L.out) return;
    const float4 bv = __ldg(reinterpret_cast<const float4*>(L.bias + o));
    const bool gelu = L.act == CFI_ACT_GELU_ERF;
    for (int rr0 = wt >> 5; rr0 < rows_per; rr0 += kSpWorkerWarps * kRows) {
        float4 t[kRows][NS];
#pragma unroll
        for (int j = 0; j < kRows; ++j) {
            const int b = split * rows_per + rr0 + j * kSpWorkerWarps;
            if (rr0 + j * kSpWorkerWarps < rows_per && b < BT && b0 + b < batch) {
                const uint32_t off = base + (uint32_t)b * 512u + (uint32_t)ch * 16u;
#pragma unroll
                for (int p = 0; p < NS; ++p)
                    t[j][p] = p == split ? *reinterpret_cast<const float4*>(smem_at(off)) : ld_cluster_f4(smem_u32(off), (uint32_t)p);
            }
        }
#pragma unroll
        for (int j = 0; j < kRows; ++j) {
            const int b = split * rows_per + rr0 + j * kSpWorkerWarps;
            if (rr0 + j * kSpWorkerWarps < rows_per && b < BT && b0 + b < batch) {
                float4 a = t[j][0];
#pragma unroll
                for (int p = 1; p < NS; ++p) a.x += t[j][p].x, a.y += t[j][p].y, a.z += t[j][p].z, a.w += t[j][p].w;
                a.x += bv.x, a.y += bv.y, a.z += bv.z, a.w += bv.w;
                if (gelu) {
                    a.x = activate(a.x, CFI_ACT_GELU_ERF);
                    a.y = activate(a.y, CFI_ACT_GELU_ERF);
                    a.z = activate(a.z, CFI_ACT_GELU_ERF);
                    a.w = activate(a.w, CFI_ACT_GELU_ERF);
                }
                *reinterpret_cast<float4*>(y + (size_t)(b0 + b) * L.out + o) = a;
            }
        }
    }
}

// Shared memory from the first 1024-byte boundary: kSpStages stages of [Wd box | x box | x_lo]; after the main loop the
// start of it holds the partial tile when K is split.  Then
//   +0 full[8] (TMA bytes), +64 ready[8] (x_lo and w_lo written), +128 empty[8] (both issuers done), +192 accumulator
//   barrier, +200 tensor-memory base.
template <int BT>
__global__ void __launch_bounds__(kSpThreads, 1)
cfi_dense_split_kernel(DevLayer L, const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
                       float* __restrict__ y, int batch) {
    static_assert(BT % 16 == 0 && BT >= 16 && BT <= 128, "batch tile");
    constexpr int kSpStages = sp_stages(BT);
    constexpr uint32_t kXBytes = sp_x_bytes(BT), kStageBytes = sp_stage_bytes(BT);
    constexpr uint32_t kABase = kSpTmemCols - 32 * kSpStages;  // accumulators in columns 0 .. 3BT-1, w_lo stages at the top
    static_assert(3 * BT <= kABase, "tensor memory: accumulators + w_lo stages");
    static_assert(kSpStages % kSpTeams == 0 && kSpStages <= 8, "a ring slot belongs to one team; eight barriers of each kind");
    constexpr int kTeam = 32 * kSpTeamWarps;                    // threads that prepare one block
    constexpr int kVec = (BT * (kSpK / 4) + kTeam - 1) / kTeam; // 16-byte pieces of the x box per worker and block
    pdl_launch_dependents();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t base = ((smem_u32(0) + 1023u) & ~1023u) - smem_u32(0);
    const uint32_t ring = base, ctl = base + sp_data_bytes(BT);
    const uint32_t full0 = smem_u32(ctl), ready0 = smem_u32(ctl + 64), empty0 = smem_u32(ctl + 128), accum = smem_u32(ctl + 192);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_at(ctl + 200));
    const int n0 = blockIdx.x * kSpM, b0 = blockIdx.y * BT;  // first output row and first batch row of the tile
    const int k_blocks = (L.in + kSpK - 1) / kSpK;
    const int split = (int)cluster_rank(), n_split = (int)cluster_size();
    const int kb0 = (int)(((int64_t)k_blocks * split) / n_split);
    const int n_local = (int)(((int64_t)k_blocks * (split + 1)) / n_split) - kb0;

    if (tid == 0) {
        prefetch_tensormap(&map_w);
        prefetch_tensormap(&map_x);
        for (int s = 0; s < kSpStages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(ready0 + 8 * s, kSpTeamWarps);
            mbar_init(empty0 + 8 * s, 2);
        }
        mbar_init(accum, 2);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        // The weight belongs to no earlier kernel: its boxes of the first ring round are requested at once, before the
        // rest of the set-up and before the wait for the kernel ahead (each stage's barrier already expects the x box
        // as well).
        for (int i = 0; i < n_local && i < kSpStages; ++i) {
            mbar_expect_tx(full0 + 8 * i, kSpWBytes + kXBytes);
            tma_load_2d(smem_u32(ring + i * kStageBytes), &map_w, full0 + 8 * i, (kb0 + i) * kSpK, n0);
        }
    }
    if (warp == 1) {  // meanwhile another warp allocates the tensor memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(ctl + 200)), "r"(kSpTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    bool ok = true;
    int issued = 0;  // thread 0: K blocks whose boxes it has requested

    if (warp == 0 && lane == 0) {
        // ---------------------------------------------------------------- TMA producer.
        // x may belong to the kernel ahead and must not be read before that kernel is done; asking for its first boxes
        // to be brought into L2 reads nothing (L2 is where that kernel's writes land, so nothing stale can be kept),
        // and a cold x is then on chip when the wait returns.  The same for the weight boxes of the second round.
        for (int i = 0; i < n_local && i < 2 * kSpStages; ++i) {
            tma_prefetch_l2_2d(&map_x, (kb0 + i) * kSpK, b0);
            if (i >= kSpStages) tma_prefetch_l2_2d(&map_w, (kb0 + i) * kSpK, n0);
        }
        pdl_wait();
        for (int i = 0; i < n_local && ok; ++i) {
            const int s = i % kSpStages;
            const uint32_t dst = smem_u32(ring + s * kStageBytes);
            if (i >= kSpStages) {
                ok = mbar_wait(empty0 + 8 * s, (uint32_t)(i / kSpStages - 1) & 1u, kTcSpinLimit);
                if (!ok) break;
                mbar_expect_tx(full0 + 8 * s, kSpWBytes + kXBytes);
                tma_load_2d(dst, &map_w, full0 + 8 * s, (kb0 + i) * kSpK, n0);
            }
            tma_load_2d(dst + kSpWBytes, &map_x, full0 + 8 * s, (kb0 + i) * kSpK, b0);
            issued = i + 1;  // (the first ring round has no wait that could fail, so no stage is left with only its weight box)
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------------------------------------------------------- first MMA issuer: Wd x [x; x_lo], N = 2 BT.
        // (The two issuers are written out separately: a thread gets a tcgen05 instruction accepted only about every
        // 150 cycles, and any branch in this loop costs more.  A stage's "ready" barrier completes only after its
        // "full" barrier has, so one wait covers both.)
        constexpr uint32_t idesc = sp_instr_desc(2 * BT);
        for (int i = 0; i < n_local && ok; ++i) {
            const int s = i % kSpStages;
            ok = mbar_wait(ready0 + 8 * s, (uint32_t)(i / kSpStages) & 1u, kTcSpinLimit);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t st = smem_u32(ring + s * kStageBytes);
            const uint64_t dw = umma_desc_k_sw128(st), dx = umma_desc_k_sw128(st + kSpWBytes);
            umma_tf32_ss(tmem_base, dw, dx, idesc, i != 0 ? 1u : 0u);  // 8 fp32 further along K: 32 bytes of a row
            umma_tf32_ss(tmem_base, dw + 2u, dx + 2u, idesc, 1u);
            umma_tf32_ss(tmem_base, dw + 4u, dx + 4u, idesc, 1u);
            umma_tf32_ss(tmem_base, dw + 6u, dx + 6u, idesc, 1u);
            umma_commit(empty0 + 8 * s);
        }
        umma_commit(accum);  // also after a failed wait: the arrival then tells when the MMAs issued so far are done
    } else if (warp == 2 && lane == 0) {
        // ---------------------------------------------------------------- second MMA issuer: w_lo x x, N = BT
        constexpr uint32_t idesc = sp_instr_desc(BT);
        const uint32_t acc = tmem_base + (uint32_t)(2 * BT);
        for (int i = 0; i < n_local && ok; ++i) {
            const int s = i % kSpStages;
            ok = mbar_wait(ready0 + 8 * s, (uint32_t)(i / kSpStages) & 1u, kTcSpinLimit);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t dx = umma_desc_k_sw128(smem_u32(ring + s * kStageBytes + kSpWBytes));
            const uint32_t a_lo = tmem_base + kABase + (uint32_t)(32 * s);  // 8 columns of tensor memory per K step
            umma_tf32_ts(acc, a_lo, dx, idesc, i != 0 ? 1u : 0u);
            umma_tf32_ts(acc, a_lo + 8u, dx + 2u, idesc, 1u);
            umma_tf32_ts(acc, a_lo + 16u, dx + 4u, idesc, 1u);
            umma_tf32_ts(acc, a_lo + 24u, dx + 6u, idesc, 1u);
            umma_commit(empty0 + 8 * s);
        }
        umma_commit(accum);
    } else if (warp >= kSpFirstWorker) {
        // ---------------------------------------------------------------- lo parts, then the epilogue
        const int team = (warp - kSpFirstWorker) / kSpTeamWarps;
        const int wt = tid - 32 * (kSpFirstWorker + kSpTeamWarps * team);  // 0 .. 255 within the team
        const int q = warp & 3;                                            // tensor-memory lanes 32 q .. 32 q + 31
        const int half = ((warp - kSpFirstWorker) >> 2) & 1;               // which half of a weight row
        const int part = (warp - kSpFirstWorker) >> 2;                     // later: which part of the batch columns
        const int row = 32 * q + lane;                                     // output row of the tile held by this thread
        const float bias = n0 + row < L.out ? L.bias[n0 + row] : 0.0f;     // lands long before the epilogue needs it
        pdl_wait();                                                        // y may belong to the kernel before this one
        for (int i = team; i < n_local && ok; i += kSpTeams) {
            const int s = i % kSpStages;
            ok = mbar_wait(full0 + 8 * s, (uint32_t)(i / kSpStages) & 1u, kTcSpinLimit);
            if (!ok) break;
            // x_lo: same swizzled position as the x box's element, one part further on.
            const uint32_t xs = ring + s * kStageBytes + kSpWBytes;
#pragma unroll
            for (int j = 0; j < kVec; ++j) {
                const uint32_t f = (uint32_t)(wt + j * kTeam) * 16u;
                if (f < kXBytes) {
                    const float4 v = *reinterpret_cast<const float4*>(smem_at(xs + f));
                    *reinterpret_cast<float4*>(smem_at(xs + kXBytes + f)) = make_float4(tf32_lo(v.x), tf32_lo(v.y), tf32_lo(v.z), tf32_lo(v.w));
                }
            }
            // w_lo: this thread's half (16 fp32) of output row `row`, un-permuted from the swizzle, into tensor-memory
            // columns [16 half, 16 half + 16) of the stage.
            {
                const uint32_t row_off = ring + s * kStageBytes + (uint32_t)row * 128u;
                uint32_t lo[16];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float4 w4 = *reinterpret_cast<const float4*>(smem_at(row_off + (uint32_t)(((4 * half + c) ^ (row & 7)) << 4)));
                    lo[4 * c + 0] = __float_as_uint(tf32_lo(w4.x));
                    lo[4 * c + 1] = __float_as_uint(tf32_lo(w4.y));
                    lo[4 * c + 2] = __float_as_uint(tf32_lo(w4.z));
                    lo[4 * c + 3] = __float_as_uint(tf32_lo(w4.w));
                }
                tmem_st16(tmem_base + ((uint32_t)(32 * q) << 16) + kABase + (uint32_t)(32 * s + 16 * half), lo);
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes of x_lo -> visible to the MMA's reads
            __syncwarp();
            if (lane == 0) mbar_arrive(ready0 + 8 * s);
        }
        ok = __all_sync(0xffffffffu, ok);
        if (ok) ok = mbar_wait(accum, 0u, kTcSpinLimit);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        // The four warps of a lane quarter take the 16-column chunks of the tile in turn.
        if (ok && 16 * part < BT) {
            const int o = n0 + row;
            auto drain = [&](auto gelu_tag) {
                constexpr bool kGelu = decltype(gelu_tag)::value;
#pragma unroll 1
                for (int c0 = 16 * part; c0 < BT; c0 += 64) {
                    uint32_t a[3][16];
                    const uint32_t t = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)c0;
#pragma unroll
                    for (int p = 0; p < 3; ++p) tmem_ld16(t + (uint32_t)(p * BT), a[p]);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        float sum = 0.0f;
                        if (n_local > 0)  // a CTA without K blocks has issued no MMA: its accumulators hold nothing
                            sum = (__uint_as_float(a[1][e]) + __uint_as_float(a[2][e])) + __uint_as_float(a[0][e]);
                        const int b = c0 + e;
                        if (n_split > 1) {
                            // partial tile [BT][128] fp32: consecutive lanes are consecutive output rows
                            *reinterpret_cast<float*>(smem_at(base + (uint32_t)b * 512u + (uint32_t)row * 4u)) = sum;
                        } else if (o < L.out && b0 + b < batch) {
                            const float v = sum + bias;
                            y[(size_t)(b0 + b) * L.out + o] = kGelu ? activate(v, CFI_ACT_GELU_ERF) : v;
                        }
                    }
                }
            };
            if (L.act == CFI_ACT_GELU_ERF && n_split == 1) drain(std::true_type{});
            else drain(std::false_type{});
        }
    }
    if (n_split > 1) {
        // Every thread of every CTA of the cluster passes both barriers, whatever `ok` says.
        cluster_sync_all();  // the partial tiles are complete
        if (warp >= kSpFirstWorker && ok) {
            const int wt = tid - 32 * kSpFirstWorker;
            switch (n_split) {
                case 2: sp_reduce<BT, 2>(L, y, batch, n0, b0, base, split, wt); break;
                case 3: sp_reduce<BT, 3>(L, y, batch, n0, b0, base, split, wt); break;
                case 4: sp_reduce<BT, 4>(L, y, batch, n0, b0, base, split, wt); break;
                case 5: sp_reduce<BT, 5>(L, y, batch, n0, b0, base, split, wt); break;
                case 6: sp_reduce<BT, 6>(L, y, batch, n0, b0, base, split, wt); break;
                case 7: sp_reduce<BT, 7>(L, y, batch, n0, b0, base, split, wt); break;
                default: sp_reduce<BT, 8>(L, y, batch, n0, b0, base, split, wt); break;
            }
        }
        cluster_sync_all_relaxed();  // no CTA leaves while another may still read its tile
    }
    if (!ok) atomicExch(L.status, 2);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    if (__syncthreads_or(!ok)) {
        // A wait gave up somewhere in this CTA.  It must not end while a box is still on its way into its shared memory
        // (the copy would land in, and signal a barrier of, whichever CTA gets that memory next) or while an MMA still
        // works on its tensor memory: wait, again bounded, for the boxes requested and for both issuers' last commit.
        if (tid == 0) {
            for (int j = issued > kSpStages ? issued - kSpStages : 0; j < issued; ++j)
                mbar_wait(full0 + 8 * (j % kSpStages), (uint32_t)(j / kSpStages) & 1u, kTcSpinLimit);
            mbar_wait(accum, 0u, kTcSpinLimit);
        }
        __syncthreads();
    }
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kSpTmemCols) : "memory");
    }
}
