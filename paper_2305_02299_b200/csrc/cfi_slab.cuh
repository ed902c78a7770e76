// CFI_VARIANT_SLAB: a batch of a few tens of rows (tiles of 16) from the condensed arrays, with the columns of x
// divided over a thread-block cluster.
//
// Included by cfi_layer.cu after cfi_dense_tc.cuh (it uses that file's cluster helpers and the gather layout built
// for CFI_VARIANT_BATCH).
//
// Between the small-batch kernel (x whole in shared memory, at most 8 batch rows) and the tensor-core variant (which
// streams the dense copy: 67 MB for 4096 x 4096 whatever the sparsity) lies the case the paper's layer is made for:
// a modest batch on a very sparse layer, where the condensed arrays are a few MB.  Every output row may read any
// column, so a CTA that owns whole rows needs all of x for its batch tile next to it; with 16 batch rows of 4096
// columns that is 256 KB, too much for one SM and, read by every SM, 38 MB of L2 traffic per call.  Here a cluster of
// S CTAs shares a group of output rows instead: CTA s stages only the columns of its share of the layer's column
// slabs, transposed to xs[column][16] (64 bytes per column), and walks over the rows' entries that fall into those
// slabs: the gather layout stores every row's entries slab by slab, so they are one contiguous run of 32-byte quads
// (4 weights, 4 columns).  A warp takes one row at a time: its 32 lanes are 8 quad slots x 4 batch quarters, i.e. per
// entry one 16-byte shared-memory gather and 4 FMAs per lane, the weights coming straight from L2 (every row's run is
// asked into L2 with one cp.async.bulk.prefetch at the start of the kernel).  The 8 quad slots are summed with shuffles, the
// row's 16 partial sums go to shared memory, and after the hardware cluster barrier every CTA sums its share of the
// rows over the S partial tiles in rank order through distributed shared memory, adds the bias, applies the activation
// and writes y with consecutive lanes on consecutive outputs.  No flags, no workspace, a fixed order of additions.
//
// Bound: shared-memory bandwidth, 4 bytes of gathered x per FMA as in the large-batch gather kernel, or the HBM stream
// of the quads (8 bytes per entry) when the layer is dense enough; at 95 % sparsity and above mostly the staging of x
// and the launch.

constexpr int kSlabBT = 16, kSlabThreads = 512, kSlabWarps = kSlabThreads / 32, kMaxSlabSplit = 8;

__device__ __forceinline__ float ld_cluster_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

// Shared memory: xs[(ncols_max + 1)][16] fp32 (the last column is zero: pad entries point there), part[rows_pc][16],
// slot_s[rows_pc], seg_s[rows_pc][slabs of this CTA + 1].
template <typename VT>
__global__ void __launch_bounds__(kSlabThreads)
cfi_slab_kernel(DevLayer L, const VT* __restrict__ x, VT* __restrict__ y, int batch, int rows_pc, int ncols_max) {
    pdl_launch_dependents();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, bq = lane & 3;  // quad slot 0..7, batch quarter 0..3
    const int split = (int)cluster_rank(), S = (int)cluster_size();
    const int slab_lo = (int)(((int64_t)L.n_slabs * split) / S), slab_hi = (int)(((int64_t)L.n_slabs * (split + 1)) / S);
    const int col_lo = slab_lo * L.cs, ncols = max(min(slab_hi * L.cs, L.in) - col_lo, 0);
    const int o0 = blockIdx.y * rows_pc, nrows = max(min(rows_pc, L.out - o0), 0);
    const int b0 = blockIdx.z * kSlabBT, nb = min(kSlabBT, batch - b0);
    float* xs = reinterpret_cast<float*>(smem_at(0));
    float* part = xs + (size_t)(ncols_max + 1) * kSlabBT;
    const int zero_col = ncols_max;
    const int shift = sizeof(VT) == 4 ? 8 : 7;  // a stored gather offset is (column in slab) * 64 * sizeof(VT) + a bank key below that
    const float4* wq = reinterpret_cast<const float4*>(L.wq_b);
    const int stride = L.n_slabs + 1;

    // Row metadata of the group into shared memory with one round of loads: which condensed row each output row is,
    // and where its quads start in each of this CTA's slabs (an ablated row has none).  Then every row's run of quads
    // is asked into L2 at once.  None of this belongs to an earlier kernel, so it all happens before the wait.
    const int nsl = slab_hi - slab_lo;
    // x may belong to the kernel ahead and must not be read before that kernel is done; asking for this CTA's part of
    // it to be brought into L2 reads nothing (L2 is where that kernel's writes land, so nothing stale can be kept), and
    // a cold x is then on chip when the wait returns.  One request per batch row, addresses and sizes rounded to 16
    // bytes, by the threads of the last warp: a request takes the issuing thread about a microsecond, which the first
    // warps spend on the row table instead.
    if (tid >= kSlabThreads - 32 && tid - (kSlabThreads - 32) < nb && ncols > 0) {
        const int b = tid - (kSlabThreads - 32);
        const uintptr_t p0 = reinterpret_cast<uintptr_t>(x + (size_t)(b0 + b) * L.in + col_lo), p1 = p0 + (size_t)ncols * sizeof(VT);
        const uintptr_t lo = p0 & ~(uintptr_t)15, hi = min((p1 + 15) & ~(uintptr_t)15, reinterpret_cast<uintptr_t>(x + (size_t)batch * L.in) & ~(uintptr_t)15);
        if (hi > lo) prefetch_l2(reinterpret_cast<const void*>(lo), (uint32_t)(hi - lo));
    }
    // Every row's quads (all slabs: the cluster's CTAs need them between them) are asked into L2 by the first CTA of the
    // cluster, straight from the row table in global memory, while the metadata below is still on its way.
    if (split == 0)
        for (int i = tid; i < nrows; i += kSlabThreads) {
            const int r = L.slot[o0 + i];
            if (r >= 0) prefetch_l2(wq + (size_t)r * L.stride_q * 2, (uint32_t)L.stride_q * 32u);
        }
    int32_t* slot_s = reinterpret_cast<int32_t*>(part + (size_t)rows_pc * kSlabBT);
    int32_t* seg_s = slot_s + rows_pc;  // [rows_pc][nsl + 1]
    {
        // Four loads in flight per thread, then their stores: one trip to memory for the whole table, not one per entry.
        const int n_meta = nrows * (nsl + 2);  // per row: nsl + 1 slab boundaries, then the condensed row number
        for (int e0 = tid; e0 < n_meta; e0 += 4 * kSlabThreads) {
            int32_t v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int e = e0 + u * kSlabThreads, i = e / (nsl + 2), j = e % (nsl + 2);
                v[u] = e >= n_meta ? 0 : j == nsl + 1 ? L.slot[o0 + i] : L.seg[(size_t)(o0 + i) * stride + slab_lo + j];
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int e = e0 + u * kSlabThreads, i = e / (nsl + 2), j = e % (nsl + 2);
                if (e < n_meta) {
                    if (j == nsl + 1) slot_s[i] = v[u];
                    else seg_s[i * (nsl + 1) + j] = v[u];
                }
            }
        }
    }
    __syncthreads();
    pdl_wait();  // x and y may belong to the kernel before this one

    // Stage x[b0 .. b0+15][col_lo .. col_lo+ncols) as xs[column][16]: a thread takes two columns at a time, 32 loads
    // (each coalesced across the warp) issued before the eight 16-byte stores.  The four 16-byte quarters of a column
    // are stored at quarter ^ ((column >> 1) & 3): consecutive columns are 64 bytes apart, and without this a warp's
    // stores would all fall into two groups of four banks.
    for (int c = tid; c < ncols; c += 2 * kSlabThreads) {
        float v[2][kSlabBT];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int b = 0; b < kSlabBT; ++b)
                v[u][b] = (b < nb && c + u * kSlabThreads < ncols) ? to_f32(x[(size_t)(b0 + b) * L.in + col_lo + c + u * kSlabThreads]) : 0.0f;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int cc = c + u * kSlabThreads;
            if (cc < ncols) {
#pragma unroll
                for (int qd = 0; qd < 4; ++qd)
                    *reinterpret_cast<float4*>(xs + (size_t)cc * kSlabBT + 4 * (qd ^ ((cc >> 1) & 3))) =
                        make_float4(v[u][4 * qd], v[u][4 * qd + 1], v[u][4 * qd + 2], v[u][4 * qd + 3]);
            }
        }
    }
    if (tid < kSlabBT) xs[(size_t)zero_col * kSlabBT + tid] = 0.0f;
    __syncthreads();

    for (int o = o0 + warp; o < o0 + nrows; o += kSlabWarps) {
        float a0 = 0.0f, a1 = 0.0f, a2 = 0.0f, a3 = 0.0f;
        const int r = slot_s[o - o0];
        if (r >= 0) {
            const int32_t* sg = seg_s + (o - o0) * (nsl + 1);
            const float4* row = wq + (size_t)r * L.stride_q * 2;
            // The row's quads of all this CTA's slabs are one run [sg[0], sg[nsl]): the 8 slots walk it together, so
            // a row costs one trip to L2 per 8 quads, and each slot finds its quad's slab from the run's boundaries.
            const int q_end = sg[nsl];
            int sl = 0, q = sg[0] + g;
            float4 w = make_float4(0.f, 0.f, 0.f, 0.f), wn = w;
            int4 c = make_int4(0, 0, 0, 0), cn = c;
            if (q < q_end) {
                w = __ldg(row + 2 * q);
                c = __ldg(reinterpret_cast<const int4*>(row + 2 * q + 1));
            }
            while (q < q_end) {
                const int qn = q + 8;
                if (qn < q_end) {  // the next quad of this slot is requested before this one is used
                    wn = __ldg(row + 2 * qn);
                    cn = __ldg(reinterpret_cast<const int4*>(row + 2 * qn + 1));
                }
                while (q >= sg[sl + 1]) ++sl;
                const int base = sl * L.cs;
                const float wv[4] = {w.x, w.y, w.z, w.w};
                const int cv[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int cl = cv[e] >> shift;                       // column within the slab; == cs for a pad entry
                    const int col = cl >= L.cs ? zero_col : base + cl;
                    const float4 v = *reinterpret_cast<const float4*>(xs + (size_t)col * kSlabBT + 4 * (bq ^ ((col >> 1) & 3)));
                    a0 = fmaf(wv[e], v.x, a0);
                    a1 = fmaf(wv[e], v.y, a1);
                    a2 = fmaf(wv[e], v.z, a2);
                    a3 = fmaf(wv[e], v.w, a3);
                }
                q = qn, w = wn, c = cn;
            }
        }
#pragma unroll
        for (int m = 4; m < 32; m <<= 1) {  // over the 8 quad slots
            a0 += __shfl_xor_sync(0xffffffffu, a0, m);
            a1 += __shfl_xor_sync(0xffffffffu, a1, m);
            a2 += __shfl_xor_sync(0xffffffffu, a2, m);
            a3 += __shfl_xor_sync(0xffffffffu, a3, m);
        }
        if (g == 0) *reinterpret_cast<float4*>(part + (size_t)(o - o0) * kSlabBT + 4 * bq) = make_float4(a0, a1, a2, a3);
    }

    // Every thread of every CTA of the cluster passes both barriers.
    if (S > 1) cluster_sync_all();
    else __syncthreads();
    {
        // Rows [rlo, rhi) of the group: sum over the cluster in rank order, bias, activation, store; consecutive
        // threads take consecutive output rows of one batch row.
        const int rlo = (int)(((int64_t)nrows * split) / S), cnt = (int)(((int64_t)nrows * (split + 1)) / S) - rlo;
        const uint32_t part_addr = smem_u32((uint32_t)((size_t)(ncols_max + 1) * kSlabBT * 4));
        for (int i = tid; i < cnt * nb; i += kSlabThreads) {
            const int ol = rlo + i % cnt, b = i / cnt;
            float t[kMaxSlabSplit];  // all loads issued before the first sum: one trip through distributed shared memory
#pragma unroll
            for (int p = 0; p < kMaxSlabSplit; ++p)
                if (p < S) t[p] = p == split ? part[ol * kSlabBT + b] : ld_cluster_f32(part_addr + (uint32_t)(ol * kSlabBT + b) * 4u, (uint32_t)p);
            float sum = t[0];
#pragma unroll
            for (int p = 1; p < kMaxSlabSplit; ++p)
                if (p < S) sum += t[p];
            from_f32(&y[(size_t)(b0 + b) * L.out + o0 + ol], activate(sum + L.bias[o0 + ol], L.act));
        }
    }
    if (S > 1) cluster_sync_all_relaxed();  // no CTA leaves while another may still read its partial sums
}
