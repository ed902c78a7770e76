// Device side of the library: layer construction, the forward kernels and their launch logic.
//
// Up to three device layouts are built from the caller's condensed arrays (values / column indices, both
// n_active x k, as in the paper's appendix "Condensed matrix multiplication"); the dense copy for the tensor-core
// variants is the third (see cfi_dense_tc.cuh and cfi_dense_split.cuh):
//
//   small-batch ("split-k") layout: columns stored in 16 bits for long index streams of layers narrower than 65,536
//     inputs, else in 32; rows padded to a multiple of 8 entries (4 for fp32 values with 32-bit columns) so that
//     every lane reads whole 16-byte vectors; a pad entry has weight 0 and points at one extra zero
//     element behind the staged x, so it contributes exactly 0 even when x holds inf or NaN.
//
//   large-batch layout: columns are cut into slabs that fit shared memory; each row's entries are
//     grouped by slab (sorting a row by column makes the groups contiguous), every group is padded
//     to a multiple of 4, and columns are stored relative to the slab start.  Entries are stored as
//     32-byte "quads" (4 weights, 4 columns); seg[r][s] is the first quad of row r in slab s.
#include "cfi.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <new>
#include <numeric>
#include <vector>

namespace {

constexpr int kBatchTile = 64;            // batch columns per CTA in the large-batch kernel
constexpr int kBatchSmemBudget = 216 * 1024;  // what the large-batch kernel may use of the SM's shared memory

struct DevLayer {
    const void* values;      // [n_active][kp]  fp32 or bf16
    const void* indices;     // [n_active][kp] uint16 when in_features < 65536 (idx16), else int32
    const void* wq_b;        // [n_active][stride_q] quads: 4 fp32 weights, then 4 int32 gather offsets: the byte
                             //   offset of the slab-relative column in the staged slab with the bank permutation
                             //   key folded in (a pad entry has weight 0 and points at column cs, all zero)
    const int32_t* seg;      // [out][n_slabs + 1] first quad of every slab within the output row's condensed row
    const float* bias;       // [out]
    const int32_t* slot;     // [out] -> row of the condensed arrays, or -1 if ablated
    int32_t* status;
    int in, out, n_active, k, kp, act;
    int cs, n_slabs, stride_q, maxq;  // slab width, slabs, quads per row, most quads of a row in one slab
    int idx16;                        // 1 if `indices` holds 16-bit columns
    int identity_rows;                // 1 if output row o is condensed row o for every o (no ablated row, rows in order)
};

}  // namespace

struct cfi_layer {
    DevLayer d{};
    int dtype = 0, device = 0, sm_count = 0, smem_optin = 0;
    int64_t device_bytes = 0, bytes_small = 0, bytes_gather = 0, bytes_dense = 0;
    int layouts = 0;  // CFI_LAYOUT_* bits of the device layouts that exist
    // The condensed arrays as given, each row sorted by column, kept so that further layouts can be built later.
    std::vector<float> h_values;
    std::vector<int32_t> h_cols, h_rows, h_slot;
    std::vector<void*> allocs;
    void* stage_x = nullptr;
    void* stage_y = nullptr;
    int staged_batch = 0;
    // Tensor-core variant (layers whose shapes TMA can address): dense copy of the weight and its tensor map.
    const void* w_dense = nullptr;
    int out_pad = 0;
    bool tc_ok = false;
    CUtensorMap map_w{};       // dense copy in boxes of 128 rows x 128 bytes
    CUtensorMap map_w_wide{};  // bf16 layers: boxes of 256 rows for the persistent kernel's wide tiles
};

struct cfi_stack {
    std::vector<cfi_layer*> layers;
    void* buf[2] = {nullptr, nullptr};
    int max_batch = 0, dtype = 0;
};

namespace {

// ------------------------------------------------------------------------------------------------
// device helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void from_f32(float* p, float v) { *p = v; }
__device__ __forceinline__ void from_f32(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

// Exact GELU v * Phi(v), the erf form.
__device__ __forceinline__ float activate(float v, int act) {
    return act == CFI_ACT_GELU_ERF ? 0.5f * v * (1.0f + erff(v * 0.70710678118654752f)) : v;
}

// ------------------------------------------------------------------------------------------------
// CFI_VARIANT_SIMPLE: Algorithm 1's loop nest with one thread per (b, o).  Reads the split-k layout.
// ------------------------------------------------------------------------------------------------
template <typename VT>
__global__ void cfi_simple_kernel(DevLayer L, const VT* __restrict__ x, VT* __restrict__ y, int batch) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= (int64_t)batch * L.out) return;
    const int b = (int)(t / L.out), o = (int)(t % L.out);
    const int r = L.slot[o];
    float s = 0.0f;
    if (r >= 0) {
        const VT* w = reinterpret_cast<const VT*>(L.values) + (size_t)r * L.kp;
        const size_t ix0 = (size_t)r * L.kp;
        const VT* xr = x + (size_t)b * L.in;
        for (int j = 0; j < L.kp; ++j) {  // pad entries (column == in) may sit anywhere in the row
            const int c = L.idx16 ? (int)static_cast<const uint16_t*>(L.indices)[ix0 + j] : static_cast<const int32_t*>(L.indices)[ix0 + j];
            if (c < L.in) s = fmaf(to_f32(w[j]), to_f32(xr[c]), s);
        }
    }
    from_f32(&y[t], activate(s + L.bias[o], L.act));
}

// ------------------------------------------------------------------------------------------------
// CFI_VARIANT_SPLITK: small batch.  G lanes share one output row and split its k terms; the CTA's
// x rows sit in shared memory as xs[column][BT] (+ one zero column for pad entries).
// ------------------------------------------------------------------------------------------------
// Units a lane of the split-k kernel keeps in flight: 4, or 2 of the 48-byte units of fp32 values with 16-bit columns
// (the same lanes per row, and so the same launch shapes, as 4 units of 4 entries would give).
__host__ __device__ constexpr int splitk_units_in_flight(bool fp32_values, bool idx16) { return fp32_values && idx16 ? 2 : 4; }

// One lane's unit of the weight stream: VEC weights and their VEC columns, read with 16-byte loads.  With 16-bit
// columns (every layer narrower than 65,536 inputs) a unit is 8 entries for both storage types: the index stream is
// then 2 bytes per entry instead of 4, a quarter (fp32) to a third (bf16) fewer bytes from HBM per call.
template <typename VT, bool I16> struct Chunk;

template <> struct Chunk<float, false> {  // 4 weights + 4 int32 columns
    static constexpr int VEC = 4;
    float4 w;
    int4 c;
    __device__ __forceinline__ void load(const void* values, const void* indices, size_t row_off, int v, bool pred, int pad_col) {
        if (pred) {
            w = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(values) + row_off) + v);
            c = __ldg(reinterpret_cast<const int4*>(reinterpret_cast<const int32_t*>(indices) + row_off) + v);
        } else {
            w = make_float4(0.f, 0.f, 0.f, 0.f);
            c = make_int4(pad_col, pad_col, pad_col, pad_col);
        }
    }
    __device__ __forceinline__ float weight(int e) const { return e == 0 ? w.x : e == 1 ? w.y : e == 2 ? w.z : w.w; }
    __device__ __forceinline__ int col(int e) const { return e == 0 ? c.x : e == 1 ? c.y : e == 2 ? c.z : c.w; }
};

template <> struct Chunk<__nv_bfloat16, false> {  // 8 weights + 8 int32 columns
    static constexpr int VEC = 8;
    uint4 w;
    int4 c0, c1;
    __device__ __forceinline__ void load(const void* values, const void* indices, size_t row_off, int v, bool pred, int pad_col) {
        if (pred) {
            w = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(values) + row_off) + v);
            c0 = __ldg(reinterpret_cast<const int4*>(reinterpret_cast<const int32_t*>(indices) + row_off) + 2 * v);
            c1 = __ldg(reinterpret_cast<const int4*>(reinterpret_cast<const int32_t*>(indices) + row_off) + 2 * v + 1);
        } else {
            w = make_uint4(0u, 0u, 0u, 0u);
            c0 = c1 = make_int4(pad_col, pad_col, pad_col, pad_col);
        }
    }
    __device__ __forceinline__ float weight(int e) const {
        const uint32_t u = (e >> 1) == 0 ? w.x : (e >> 1) == 1 ? w.y : (e >> 1) == 2 ? w.z : w.w;
        return (e & 1) ? bf16_hi(u) : bf16_lo(u);
    }
    __device__ __forceinline__ int col(int e) const {
        const int4& q = e < 4 ? c0 : c1;
        const int f = e & 3;
        return f == 0 ? q.x : f == 1 ? q.y : f == 2 ? q.z : q.w;
    }
};

__device__ __forceinline__ int col16(const uint4& c, int e) {
    const uint32_t u = (e >> 1) == 0 ? c.x : (e >> 1) == 1 ? c.y : (e >> 1) == 2 ? c.z : c.w;
    return (int)((e & 1) ? (u >> 16) : (u & 0xFFFFu));
}

template <> struct Chunk<float, true> {  // 8 weights + 8 uint16 columns
    static constexpr int VEC = 8;
    float4 w0, w1;
    uint4 c;
    __device__ __forceinline__ void load(const void* values, const void* indices, size_t row_off, int v, bool pred, int pad_col) {
        if (pred) {
            w0 = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(values) + row_off) + 2 * v);
            w1 = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(values) + row_off) + 2 * v + 1);
            c = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(indices) + row_off) + v);
        } else {
            w0 = w1 = make_float4(0.f, 0.f, 0.f, 0.f);
            const uint32_t p = (uint32_t)pad_col | ((uint32_t)pad_col << 16);
            c = make_uint4(p, p, p, p);
        }
    }
    __device__ __forceinline__ float weight(int e) const {
        const float4& q = e < 4 ? w0 : w1;
        const int f = e & 3;
        return f == 0 ? q.x : f == 1 ? q.y : f == 2 ? q.z : q.w;
    }
    __device__ __forceinline__ int col(int e) const { return col16(c, e); }
};

template <> struct Chunk<__nv_bfloat16, true> {  // 8 weights + 8 uint16 columns
    static constexpr int VEC = 8;
    uint4 w, c;
    __device__ __forceinline__ void load(const void* values, const void* indices, size_t row_off, int v, bool pred, int pad_col) {
        if (pred) {
            w = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(values) + row_off) + v);
            c = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(indices) + row_off) + v);
        } else {
            w = make_uint4(0u, 0u, 0u, 0u);
            const uint32_t p = (uint32_t)pad_col | ((uint32_t)pad_col << 16);
            c = make_uint4(p, p, p, p);
        }
    }
    __device__ __forceinline__ float weight(int e) const {
        const uint32_t u = (e >> 1) == 0 ? w.x : (e >> 1) == 1 ? w.y : (e >> 1) == 2 ? w.z : w.w;
        return (e & 1) ? bf16_hi(u) : bf16_lo(u);
    }
    __device__ __forceinline__ int col(int e) const { return col16(c, e); }
};

template <int BT>
__device__ __forceinline__ void gather_fma(float (&acc)[BT], const float* xs, int col, float w) {
    const float* p = xs + (size_t)col * BT;
    if constexpr (BT == 1) {
        acc[0] = fmaf(w, p[0], acc[0]);
    } else if constexpr (BT == 2) {
        const float2 v = *reinterpret_cast<const float2*>(p);
        acc[0] = fmaf(w, v.x, acc[0]);
        acc[1] = fmaf(w, v.y, acc[1]);
    } else {
#pragma unroll
        for (int q = 0; q < BT / 4; ++q) {
            const float4 v = *reinterpret_cast<const float4*>(p + 4 * q);
            acc[4 * q + 0] = fmaf(w, v.x, acc[4 * q + 0]);
            acc[4 * q + 1] = fmaf(w, v.y, acc[4 * q + 1]);
            acc[4 * q + 2] = fmaf(w, v.z, acc[4 * q + 2]);
            acc[4 * q + 3] = fmaf(w, v.w, acc[4 * q + 3]);
        }
    }
}

// Programmatic dependent launch.  Every forward kernel lets its successor in the stream start early
// (pdl_launch_dependents at its top) and itself touches x and y only after pdl_wait, which returns once the
// predecessor has completed and its writes are visible.  What a kernel does before pdl_wait (reading the
// layer's weights, indices and tables, which no kernel writes) therefore overlaps the predecessor's tail.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Ask for `bytes` (a multiple of 16, from a 16-byte aligned address) to be brought into L2.  Costs one
// instruction and no registers; later loads of the range then find it on chip.
__device__ __forceinline__ void prefetch_l2(const void* p, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

// A lane keeps U units (16-byte vectors of weights with their indices) in flight in registers; the rest of the row is
// on its way into L2.  XS = loads of x in flight per thread while staging (8 where few threads stage a long x).
template <typename VT, bool I16, int BT, int G, int XS>
__global__ void __launch_bounds__(512) cfi_splitk_kernel(DevLayer L, const VT* __restrict__ x, VT* __restrict__ y, int batch,
                                  int rows_per_group) {
    extern __shared__ __align__(16) float xs_f32[];  // [(in + 1)][BT]
    float* xs = xs_f32;
    using CK = Chunk<VT, I16>;
    constexpr uint32_t kIdxBytes = I16 ? 2 : 4;
    constexpr int U = splitk_units_in_flight(sizeof(VT) == 4, I16);
    pdl_launch_dependents();
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int b0 = blockIdx.y * BT;
    const int nb = min(BT, batch - b0);
    const int groups = nthr / G, g = tid / G, lg = tid % G;
    const int nvec = L.kp / CK::VEC;
    const bool dense_rows = L.identity_rows != 0;  // output row o is condensed row o: no look-up through slot[]
    int o = blockIdx.x * (groups * rows_per_group) + g;
    int r = o < L.out ? (dense_rows ? o : L.slot[o]) : -1;

    // The first row's weights and indices depend neither on x nor on the kernel before this one.  The whole row
    // is asked into L2 by one lane, and its first vectors are requested into registers, before anything else,
    // so the weight stream is in flight while x is awaited and staged.
    const bool long_row = nvec > G * U;  // else the first units of the lanes are the whole row: nothing left to ask for
    if (lg == 0 && r >= 0 && long_row) {
        prefetch_l2(reinterpret_cast<const VT*>(L.values) + (size_t)r * L.kp, (uint32_t)(L.kp * sizeof(VT)));
        prefetch_l2(static_cast<const unsigned char*>(L.indices) + (size_t)r * L.kp * kIdxBytes, (uint32_t)L.kp * kIdxBytes);
    }
    CK ck[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int v = lg + u * G;
        ck[u].load(L.values, L.indices, (size_t)max(r, 0) * L.kp, v, r >= 0 && v < nvec, L.in);
    }
    float bias = o < L.out ? L.bias[o] : 0.0f;
    // x may belong to the kernel ahead and must not be read before that kernel is done; asking for it to be brought
    // into L2 reads nothing (L2 is where that kernel's writes land, so nothing stale can be kept), and a cold x is
    // then on chip when the wait returns.  The first CTAs of a batch tile ask, 16 KB per thread.
    if (blockIdx.x < 2 && ((size_t)L.in * sizeof(VT)) % 16 == 0) {
        const size_t bytes = (size_t)nb * L.in * sizeof(VT), off = (size_t)tid << 14;
        if (off < bytes)
            prefetch_l2(reinterpret_cast<const unsigned char*>(x + (size_t)b0 * L.in) + off, (uint32_t)min(bytes - off, (size_t)1 << 14));
    }

    pdl_wait();
    // Stage the CTA's x rows, widened to fp32, transposed to [column][b].  Loads are issued kXStage at a time
    // before their stores, so staging costs a few memory round trips, not one per element.
    constexpr int kXStage = XS;
    if (BT == 1 && sizeof(VT) == 4 && (L.in & 3) == 0) {
        const float4* src = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(x) + (size_t)b0 * L.in);
        const int n4 = L.in >> 2;
        for (int c0 = tid; c0 < n4; c0 += nthr * kXStage) {
            float4 v[kXStage];
#pragma unroll
            for (int u = 0; u < kXStage; ++u)
                if (c0 + u * nthr < n4) v[u] = __ldg(src + c0 + u * nthr);
#pragma unroll
            for (int u = 0; u < kXStage; ++u)
                if (c0 + u * nthr < n4) reinterpret_cast<float4*>(xs)[c0 + u * nthr] = v[u];
        }
    } else {
        // A thread takes kCols columns at a time: one load per column and batch row (each coalesced across the
        // warp), all issued before the first store, then each column's BT values go to shared memory side by side.
        constexpr int kCols = BT >= 8 ? 4 : BT >= 4 ? 4 : 8;
        for (int c0 = tid; c0 < L.in; c0 += nthr * kCols) {
            float v[kCols][BT];
#pragma unroll
            for (int u = 0; u < kCols; ++u)
#pragma unroll
                for (int b = 0; b < BT; ++b)
                    v[u][b] = (b < nb && c0 + u * nthr < L.in) ? to_f32(x[(size_t)(b0 + b) * L.in + c0 + u * nthr]) : 0.0f;
#pragma unroll
            for (int u = 0; u < kCols; ++u) {
                const int c = c0 + u * nthr;
                if (c < L.in) {
                    if constexpr (BT == 1) {
                        xs[c] = v[u][0];
                    } else if constexpr (BT == 2) {
                        *reinterpret_cast<float2*>(xs + (size_t)c * 2) = make_float2(v[u][0], v[u][1]);
                    } else {
#pragma unroll
                        for (int q = 0; q < BT / 4; ++q)
                            *reinterpret_cast<float4*>(xs + (size_t)c * BT + 4 * q) =
                                make_float4(v[u][4 * q], v[u][4 * q + 1], v[u][4 * q + 2], v[u][4 * q + 3]);
                    }
                }
            }
        }
    }
    if (tid < BT) xs[(size_t)L.in * BT + tid] = 0.0f;
    __syncthreads();

    for (int i = 0;;) {
        float acc[BT];
#pragma unroll
        for (int b = 0; b < BT; ++b) acc[b] = 0.0f;
        if (r >= 0) {
            const size_t row_off = (size_t)r * L.kp;
            for (int v0 = lg;;) {
#pragma unroll
                for (int u = 0; u < U; ++u)
#pragma unroll
                    for (int e = 0; e < CK::VEC; ++e) gather_fma<BT>(acc, xs, ck[u].col(e), ck[u].weight(e));
                v0 += G * U;
                if (v0 >= nvec) break;
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int v = v0 + u * G;
                    ck[u].load(L.values, L.indices, row_off, v, v < nvec, L.in);
                }
            }
        }
        const int o_done = o;
        const float bias_done = bias;
        // The next row's first vectors and bias are requested before this row's reduction and store.
        const bool more = ++i < rows_per_group;
        if (more) {
            o += groups;
            r = o < L.out ? (dense_rows ? o : L.slot[o]) : -1;
            if (lg == 0 && r >= 0 && long_row) {
                prefetch_l2(reinterpret_cast<const VT*>(L.values) + (size_t)r * L.kp, (uint32_t)(L.kp * sizeof(VT)));
                prefetch_l2(static_cast<const unsigned char*>(L.indices) + (size_t)r * L.kp * kIdxBytes, (uint32_t)L.kp * kIdxBytes);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = lg + u * G;
                ck[u].load(L.values, L.indices, (size_t)max(r, 0) * L.kp, v, r >= 0 && v < nvec, L.in);
            }
            bias = o < L.out ? L.bias[o] : 0.0f;
        }
        // Finish the k-sum across the G lanes of the group.
#pragma unroll
        for (int b = 0; b < BT; ++b) {
            float v = acc[b];
#pragma unroll
            for (int m = G >> 1; m > 0; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
            acc[b] = v;
        }
        if (lg == 0 && o_done < L.out) {
#pragma unroll
            for (int b = 0; b < BT; ++b)
                if (b < nb) from_f32(&y[(size_t)(b0 + b) * L.out + o_done], activate(acc[b] + bias_done, L.act));
        }
        if (!more) break;
    }
}

// ------------------------------------------------------------------------------------------------
// CFI_VARIANT_BATCH: large batch.  A CTA owns a tile of `rt` consecutive output rows x BT batch columns
// and walks the columns of x slab by slab.  Two shared-memory buffers hold x slabs transposed,
// xs[column][BT], so that one column index yields BT contiguous batch values.
//
// Warps are split into row groups of BT/4 lanes.  A group owns RPH rows of the tile and keeps their
// partial sums in registers across slabs.  Work proceeds in items (slab s, row j of the group):
//   - the row's quads of the NEXT item (4 weights + 4 gather offsets = 32 bytes each) are copied into a
//     warp-private buffer with cp.async;
//   - the thread's share of the NEXT slab of x, a 4 x 4 block, is requested from global memory (16 bytes
//     per lane and batch row, whole 128-byte lines per row and warp);
//   - the current item is computed: per entry one 16-byte (fp32) or 8-byte (bf16) shared-memory gather
//     of the lane's 4 batch values and 4 FMAs;
//   - the block requested above is transposed in registers and stored into the other buffer.
// One __syncthreads per slab publishes the next buffer.  Global latency is thus hidden behind an item's
// arithmetic by every warp, and no warp is reserved for data movement.  At the end the sums go through
// shared memory once more so that y[b, o] is written in runs of consecutive o.
//
// Within a staged column the BT/4 four-value units are permuted by unit ^ ((column / 4) & (BT/4 - 1)).
// The staging stores (one unit per lane) then fall into distinct banks within every quarter warp, and a
// reading row group still sees consecutive units in distinct banks.  The layer
// stores, per entry, the byte offset of its column with the permutation key folded in, so a lane's
// gather address is that offset XOR (its unit number * unit bytes).
//
// All shared-memory addresses are 32-bit byte offsets from the start of the dynamic shared memory.
// ------------------------------------------------------------------------------------------------
constexpr int kMaxRowsPerGroup = 8;
constexpr int kStageUnroll = 2;  // 4 x 4 blocks (4 loads each) in flight per thread outside the row items

// Dynamic shared memory as bytes; every extern __shared__ array starts at the same address.
__device__ __forceinline__ unsigned char* smem_at(uint32_t off) {
    extern __shared__ __align__(128) unsigned char smem_dyn[];
    return smem_dyn + off;
}

__device__ __forceinline__ void cp_async16(uint32_t smem_off, const void* gmem_src) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_at(smem_off));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// One gather + 4 FMAs.  addr = buffer offset + (entry's stored offset XOR the lane's unit offset).
template <typename VT>
__device__ __forceinline__ void fma4(float (&a)[4], uint32_t addr, float w);
template <>
__device__ __forceinline__ void fma4<float>(float (&a)[4], uint32_t addr, float w) {
    const float4 v = *reinterpret_cast<const float4*>(smem_at(addr));
    a[0] = fmaf(w, v.x, a[0]);
    a[1] = fmaf(w, v.y, a[1]);
    a[2] = fmaf(w, v.z, a[2]);
    a[3] = fmaf(w, v.w, a[3]);
}
template <>
__device__ __forceinline__ void fma4<__nv_bfloat16>(float (&a)[4], uint32_t addr, float w) {
    const uint2 v = *reinterpret_cast<const uint2*>(smem_at(addr));
    a[0] = fmaf(w, bf16_lo(v.x), a[0]);
    a[1] = fmaf(w, bf16_hi(v.x), a[1]);
    a[2] = fmaf(w, bf16_lo(v.y), a[2]);
    a[3] = fmaf(w, bf16_hi(v.y), a[3]);
}

// Shared-memory carve-up, identical on host and device.
struct BatchSmem {
    uint32_t xs_bytes;  // one x buffer
    uint32_t meta_off;  // slot_s[rt], bias_s[rt], seg_s[rt][n_slabs + 1]
    uint32_t wbuf_off;  // [warp][2 stages][row groups per warp][maxq] quads of 32 bytes
    size_t total;
};
__host__ __device__ inline BatchSmem batch_smem_layout(int cs, int n_slabs, int maxq, int elem, int bt, int rt,
                                                       int warps) {
    BatchSmem m;
    m.xs_bytes = (uint32_t)((((size_t)(cs + 1) * bt * elem) + 127) & ~(size_t)127);
    m.meta_off = 2 * m.xs_bytes;
    const uint32_t meta = (uint32_t)((((size_t)rt * (n_slabs + 3) * 4) + 31) & ~(size_t)31);
    m.wbuf_off = m.meta_off + meta;
    m.total = (size_t)m.wbuf_off + (size_t)warps * 2 * (128 / bt) * maxq * 32;
    return m;
}

// x staging.  A "warp block" wb is 16 batch rows x 32 consecutive columns of a slab.  Lane = (cl, uq): it reads
// the 4 columns c..c+3 (c = 32 * (wb / (BT/16)) + 4 * cl) of the 4 batch rows of unit u, one 16-byte (fp32) or
// 8-byte (bf16) load per row, transposes the 4 x 4 block in registers and writes column c + j's 4 batch values
// with one 16-byte / 8-byte store to unit u ^ key(c).  Per load instruction a warp reads 128 contiguous bytes
// of 4 batch rows; per store instruction every quarter (fp32) or half (bf16) of the warp hits distinct banks.
template <typename VT, int BT>
struct Stager {
    const VT* x;   // &x[b0][c0]: first batch row of the tile, first column of the slab
    int in, cl, uq, nb, ncol;
    bool vec_ok;
    struct alignas(16) Block { VT v[4][4]; };  // [batch row in unit][column in chunk]

    __device__ __forceinline__ int unit_of(int wb) const { return ((uq & 1) * 8 + (uq >> 1) * 4 + (wb & 3)) & (BT / 4 - 1); }

    __device__ __forceinline__ void load(int wb, int n_blocks, Block& blk) const {
        static_assert(BT == 64, "lane mapping assumes 16 units per staged column");
        const int u = unit_of(wb), c = ((wb >> 2) * 8 + cl) * 4;
        const bool live = wb < n_blocks;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int b = 4 * u + i;
            const VT* src = x + (size_t)b * in + c;
            if (live && b < nb && vec_ok && c + 3 < ncol) {
                if constexpr (sizeof(VT) == 4) {
                    const float4 t = __ldg(reinterpret_cast<const float4*>(src));
                    blk.v[i][0] = t.x, blk.v[i][1] = t.y, blk.v[i][2] = t.z, blk.v[i][3] = t.w;
                } else {
                    *reinterpret_cast<uint2*>(blk.v[i]) = __ldg(reinterpret_cast<const uint2*>(src));
                }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) blk.v[i][j] = (live && b < nb && c + j < ncol) ? src[j] : VT(0.0f);
            }
        }
    }
    // xs_off: byte offset of the destination buffer.
    __device__ __forceinline__ void store(int wb, uint32_t xs_off, const Block& blk) const {
        const int u = unit_of(wb), c = ((wb >> 2) * 8 + cl) * 4;
        constexpr uint32_t unit_bytes = 4 * sizeof(VT), col_bytes = BT * sizeof(VT);
        const uint32_t base = xs_off + (uint32_t)c * col_bytes + (uint32_t)(u ^ ((c >> 2) & (BT / 4 - 1))) * unit_bytes;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (c + j < ncol) {
                if constexpr (sizeof(VT) == 4) {
                    *reinterpret_cast<float4*>(smem_at(base + j * col_bytes)) =
                        make_float4(blk.v[0][j], blk.v[1][j], blk.v[2][j], blk.v[3][j]);
                } else {
                    const uint32_t* w0 = reinterpret_cast<const uint32_t*>(blk.v[0]);
                    const uint32_t* w1 = reinterpret_cast<const uint32_t*>(blk.v[1]);
                    const uint32_t* w2 = reinterpret_cast<const uint32_t*>(blk.v[2]);
                    const uint32_t* w3 = reinterpret_cast<const uint32_t*>(blk.v[3]);
                    const uint32_t sel = (j & 1) ? 0x7632u : 0x5410u;
                    *reinterpret_cast<uint2*>(smem_at(base + j * col_bytes)) =
                        make_uint2(__byte_perm(w0[j >> 1], w1[j >> 1], sel), __byte_perm(w2[j >> 1], w3[j >> 1], sel));
                }
            }
        }
    }
};

template <typename VT, int BT, int RPH>
__global__ void __launch_bounds__(512, 1)
cfi_batch_kernel(DevLayer L, const VT* __restrict__ x, VT* __restrict__ y, int batch) {
    constexpr int LPR = BT / 4, RPW = 32 / LPR;  // lanes per row group, row groups per warp
    pdl_launch_dependents();
    const int tid = threadIdx.x, nthr = blockDim.x, warp = tid >> 5, lane = tid & 31;
    const int nwarps = nthr >> 5, ngroups = nwarps * RPW, rt = ngroups * RPH, S = L.n_slabs;
    const BatchSmem lay = batch_smem_layout(L.cs, S, L.maxq, (int)sizeof(VT), BT, rt, nwarps);
    int32_t* slot_s = reinterpret_cast<int32_t*>(smem_at(lay.meta_off));
    float* bias_s = reinterpret_cast<float*>(slot_s + rt);
    int32_t* seg_s = slot_s + 2 * rt;  // [rt][S + 1]
    const int b0 = blockIdx.y * BT, nb = min(BT, batch - b0);
    const int o0 = blockIdx.x * rt, nrows = min(rt, L.out - o0);

    // Tile metadata: which condensed row each output row is, where its quads start in every slab, its bias.
    for (int i = tid; i < rt; i += nthr) {
        slot_s[i] = i < nrows ? L.slot[o0 + i] : -1;
        bias_s[i] = i < nrows ? L.bias[o0 + i] : 0.0f;
    }
    for (int e = tid; e < rt * (S + 1); e += nthr) seg_s[e] = e < nrows * (S + 1) ? L.seg[(size_t)o0 * (S + 1) + e] : 0;
    if (tid < BT) {  // the zero column that pad entries point at, in both buffers
        reinterpret_cast<VT*>(smem_at(0))[(size_t)L.cs * BT + tid] = VT(0.0f);
        reinterpret_cast<VT*>(smem_at(lay.xs_bytes))[(size_t)L.cs * BT + tid] = VT(0.0f);
    }

    Stager<VT, BT> st;
    st.in = L.in, st.cl = lane & 7, st.uq = lane >> 3, st.nb = nb, st.vec_ok = (L.in & 3) == 0;
    const VT* x_tile = x + (size_t)b0 * L.in;

    // Slab 0: everybody stages, kStageUnroll blocks (4 loads each) in flight per thread.  x (and later y) may
    // belong to the kernel before this one, so this is where its completion is awaited.
    pdl_wait();
    {
        st.x = x_tile, st.ncol = min(L.cs, L.in);
        const int n_blocks = ((st.ncol + 31) >> 5) * (BT / 16);
        for (int w0 = warp; w0 < n_blocks; w0 += nwarps * kStageUnroll) {
            typename Stager<VT, BT>::Block blk[kStageUnroll];
#pragma unroll
            for (int u = 0; u < kStageUnroll; ++u) st.load(w0 + u * nwarps, n_blocks, blk[u]);
#pragma unroll
            for (int u = 0; u < kStageUnroll; ++u)
                if (w0 + u * nwarps < n_blocks) st.store(w0 + u * nwarps, 0u, blk[u]);
        }
    }
    __syncthreads();

    const int sub = lane / LPR, ll = lane % LPR;
    const uint32_t lane_key = (uint32_t)(ll * 4 * (int)sizeof(VT));
    const int g = warp * RPW + sub;  // row group within the CTA; its rows are g, g + ngroups, ...
    const uint32_t stage_bytes = (uint32_t)(RPW * L.maxq * 32);
    const uint32_t wbuf = lay.wbuf_off + (uint32_t)warp * 2 * stage_bytes + (uint32_t)sub * L.maxq * 32;
    const float4* wq = reinterpret_cast<const float4*>(L.wq_b);

    // Copy the quads of item (slab s, row j of this group) into stage `st`.  The group is committed even
    // when empty so that every lane counts the same number of groups.
    auto prefetch = [&](int s, int j, int stage) {
        const int i = g + j * ngroups;
        const int r = slot_s[i];
        if (r >= 0) {
            const int q0 = seg_s[i * (S + 1) + s], q1 = seg_s[i * (S + 1) + s + 1];
            const float4* src = wq + ((size_t)r * L.stride_q + q0) * 2;
            const uint32_t dst = wbuf + stage * stage_bytes;
            for (int ch = ll; ch < 2 * (q1 - q0); ch += LPR) cp_async16(dst + ch * 16, src + ch);
        }
        cp_async_commit();
    };

    float acc[RPH][4];
#pragma unroll
    for (int j = 0; j < RPH; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[j][e] = 0.0f;

    prefetch(0, 0, 0);
    int n = 0;
    for (int s = 0; s < S; ++s) {
        const uint32_t xs_off = (s & 1) ? lay.xs_bytes : 0u, xs_next = (s & 1) ? 0u : lay.xs_bytes;
        const int c0n = (s + 1) * L.cs;
        st.ncol = s + 1 < S ? min(L.cs, L.in - c0n) : 0;
        st.x = x_tile + c0n;
        const int n_blocks = ((st.ncol + 31) >> 5) * (BT / 16);  // warp blocks of the next slab
#pragma unroll
        for (int j = 0; j < RPH; ++j) {
            __syncwarp();  // every lane is done reading the stage the next prefetch overwrites
            const int jn = j + 1 < RPH ? j + 1 : 0, sn = j + 1 < RPH ? s : s + 1;
            if (sn < S) prefetch(sn, jn, (n + 1) & 1);
            typename Stager<VT, BT>::Block xv;  // this item's share of the next slab
            st.load(warp + j * nwarps, n_blocks, xv);
            if (sn < S) cp_async_wait<1>();
            else cp_async_wait<0>();
            __syncwarp();  // the other lanes' copies of this item are visible too
            const int i = g + j * ngroups;
            if (slot_s[i] >= 0) {
                const int nq = seg_s[i * (S + 1) + s + 1] - seg_s[i * (S + 1) + s];
                const uint32_t wb = wbuf + (n & 1) * stage_bytes;
#pragma unroll 2
                for (int q = 0; q < nq; ++q) {
                    const float4 w = *reinterpret_cast<const float4*>(smem_at(wb + q * 32));
                    const int4 c = *reinterpret_cast<const int4*>(smem_at(wb + q * 32 + 16));
                    fma4<VT>(acc[j], xs_off + ((uint32_t)c.x ^ lane_key), w.x);
                    fma4<VT>(acc[j], xs_off + ((uint32_t)c.y ^ lane_key), w.y);
                    fma4<VT>(acc[j], xs_off + ((uint32_t)c.z ^ lane_key), w.z);
                    fma4<VT>(acc[j], xs_off + ((uint32_t)c.w ^ lane_key), w.w);
                }
            }
            if (warp + j * nwarps < n_blocks) st.store(warp + j * nwarps, xs_next, xv);
            ++n;
        }
        // Whatever of the next slab the row items did not cover.
        for (int w0 = warp + RPH * nwarps; w0 < n_blocks; w0 += nwarps * kStageUnroll) {
            typename Stager<VT, BT>::Block blk[kStageUnroll];
#pragma unroll
            for (int u = 0; u < kStageUnroll; ++u) st.load(w0 + u * nwarps, n_blocks, blk[u]);
#pragma unroll
            for (int u = 0; u < kStageUnroll; ++u)
                if (w0 + u * nwarps < n_blocks) st.store(w0 + u * nwarps, xs_next, blk[u]);
        }
        __syncthreads();  // next slab is complete, and nobody reads this slab's buffer any more
    }

    // Epilogue: bias + activation, then through shared memory (ys[b][row]) so that y is written in runs of
    // consecutive output rows per batch row.
    float* ys = reinterpret_cast<float*>(smem_at(0));
    const int pitch = rt | 1;
    float bias_r[RPH];
#pragma unroll
    for (int j = 0; j < RPH; ++j) bias_r[j] = bias_s[g + j * ngroups];
    __syncthreads();  // bias_s is read; the y tile may now overwrite any part of shared memory
#pragma unroll
    for (int j = 0; j < RPH; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) ys[(4 * ll + e) * pitch + g + j * ngroups] = activate(acc[j][e] + bias_r[j], L.act);
    __syncthreads();
    const int per_b = nrows;
    for (int b = warp; b < nb; b += nwarps) {
        VT* yrow = y + (size_t)(b0 + b) * L.out + o0;
        for (int i = lane; i < per_b; i += 32) from_f32(&yrow[i], ys[b * pitch + i]);
    }
}

#include "cfi_dense_tc.cuh"
#include "cfi_slab.cuh"
#include "cfi_dense_split.cuh"
#include "cfi_dense_tc_persistent.cuh"

// ------------------------------------------------------------------------------------------------
// host: launch shapes
// ------------------------------------------------------------------------------------------------
struct SplitkShape { int bt, g, xs, threads, rows_per_group, grid_x, grid_y; size_t smem; };
struct BatchShape { int warps, rph, threads, rt, grid_x, grid_y; size_t smem; bool ok; };

// Entries per 16-byte unit of the small-batch layout: 8 for bf16 values and wherever the columns are 16-bit, else 4.
// 16-bit columns: possible when the pad column `in` is representable, worth it when the index stream is long.  They
// save 2 bytes per entry from HBM and cost a few instructions per unit on the critical path of a row; measured at
// batch 1, layers below about a million entries run at the launch floor either way and were 0.2-0.3 us slower with
// them, 4096 x 4096 at 80 % (3.4 M entries) went from 5.6 to 4.9 us.
bool use_idx16(int in_features, int64_t nnz) { return in_features < 65536 && nnz >= 1500000; }
int vec_of(int dtype, bool idx16) { return (dtype == CFI_BF16 || idx16) ? 8 : 4; }

// Lanes that share a row in the split-k kernel: the smallest power of two for which the units a lane keeps in flight
// cover the row, at most a warp.  The small-batch layout orders a row's entries for this number (order_for_banks).
int splitk_lanes_per_row(int nvec, int units) {
    int g = 4;
    while (g < 32 && g * units < nvec) g <<= 1;
    return g;
}

SplitkShape splitk_shape(const cfi_layer* l, int batch) {
    SplitkShape s{};
    s.bt = batch >= 8 ? 8 : batch >= 3 ? 4 : batch == 2 ? 2 : 1;
    while (s.bt > 1 && (size_t)(l->d.in + 1) * s.bt * 4 > (size_t)l->smem_optin) s.bt >>= 1;
    const int nvec = l->d.kp / vec_of(l->dtype, l->d.idx16 != 0);
    s.g = splitk_lanes_per_row(nvec, splitk_units_in_flight(l->dtype == CFI_F32, l->d.idx16 != 0));
    // Every CTA stages x for itself (from L2), so larger CTAs spend less of the L2 bandwidth on x.  The staged x
    // also limits how many CTAs fit an SM; the grid is sized to one wave of what fits (at most eight CTAs per
    // SM), with several rows per group when needed (rows of a group run one after the other).
    s.smem = (size_t)(l->d.in + 1) * s.bt * 4;
    const int fit = (int)std::max<size_t>(1, std::min<size_t>(8, ((size_t)227 * 1024) / (s.smem + 1024)));
    const int64_t lanes = (int64_t)l->d.out * s.g;
    s.threads = lanes >= (int64_t)l->sm_count * 256 ? 256 : 128;
    if (fit <= 2 && lanes >= (int64_t)l->sm_count * 512) s.threads = 512;
    const int groups = s.threads / s.g;
    const int ctas_one_row_each = (l->d.out + groups - 1) / groups;
    s.grid_y = (batch + s.bt - 1) / s.bt;
    const int target = std::max(1, l->sm_count * fit / s.grid_y);  // the batch tiles share the wave
    s.rows_per_group = std::max(1, (ctas_one_row_each + target - 1) / target);
    // x loads in flight per staging thread: 8 when 4 would need more than one round and the grid is small enough
    // that the extra registers do not cost a wave.
    s.xs = (l->d.in > 16 * s.threads && s.threads == 128) ? 8 : 4;
    s.grid_x = (l->d.out + groups * s.rows_per_group - 1) / (groups * s.rows_per_group);
    s.grid_y = (batch + s.bt - 1) / s.bt;
    s.smem = (size_t)(l->d.in + 1) * s.bt * 4;
    return s;
}

size_t batch_smem(const cfi_layer* l, int warps, int rph) {
    const int es = l->dtype == CFI_BF16 ? 2 : 4;
    const int rt = warps * (128 / kBatchTile) * rph;
    const BatchSmem m = batch_smem_layout(l->d.cs, l->d.n_slabs, l->d.maxq, es, kBatchTile, rt, warps);
    return std::max(m.total, (size_t)kBatchTile * (rt | 1) * 4);  // the epilogue's y tile reuses the start
}

// Tile shape: warps (6..16) and rows per row group (1..8) give rt = 2 * warps * rph rows per CTA.
// Shared-memory traffic bounds this kernel, so the cost of a CTA is counted in 128-byte wavefronts:
// gathers and weight reads per entry, the transposed staging of x, plus a fixed start-up; the grid runs
// in waves of one CTA per SM.
BatchShape batch_shape(const cfi_layer* l, int batch) {
    BatchShape best{};
    best.ok = false;
    if (!(l->layouts & CFI_LAYOUT_GATHER)) return best;
    double best_cost = 0;
    const int es = l->dtype == CFI_BF16 ? 2 : 4;
    const int grid_y = (batch + kBatchTile - 1) / kBatchTile;
    const double per_entry = kBatchTile * es / 128.0 + 0.5, staging = (double)l->d.in * kBatchTile * es / 128.0;
    for (int warps = 6; warps <= 16; ++warps)
        for (int rph = 1; rph <= kMaxRowsPerGroup; ++rph) {
            const size_t smem = batch_smem(l, warps, rph);
            if (smem > (size_t)l->smem_optin) continue;
            const int rt = warps * (128 / kBatchTile) * rph;
            const int64_t tiles = (int64_t)((l->d.out + rt - 1) / rt) * grid_y;
            const int64_t waves = (tiles + l->sm_count - 1) / l->sm_count;
            const double cost = (double)waves * ((double)rt * l->d.stride_q * 4 * per_entry + staging + 4000.0);
            if (!best.ok || cost < best_cost * 0.999 || (cost < best_cost * 1.001 && warps > best.warps)) {
                best = BatchShape{warps, rph, warps * 32, rt, (l->d.out + rt - 1) / rt, grid_y, smem, true};
                best_cost = cost;
            }
        }
    return best;
}

// ------------------------------------------------------------------------------------------------
// host: launches
// ------------------------------------------------------------------------------------------------
// Opt in to more than 48 KB of dynamic shared memory.  The attribute is per kernel and per device, so the
// largest value set so far is remembered per (kernel, device) and the runtime is only called to raise it.
constexpr int kMaxDevices = 64;

template <auto Kernel>
cfi_status_t set_smem(size_t bytes, int device) {
    static std::atomic<int> granted[kMaxDevices];
    if (bytes <= 48 * 1024) return CFI_OK;
    const bool tracked = device >= 0 && device < kMaxDevices;
    if (tracked && granted[device].load(std::memory_order_relaxed) >= (int)bytes) return CFI_OK;
    if (cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
        cudaGetLastError();
        return CFI_ERR_SHAPE;
    }
    if (tracked) granted[device].store((int)bytes, std::memory_order_relaxed);
    return CFI_OK;
}

// Launch with programmatic stream serialisation allowed: the kernel may start before its predecessor in the
// stream has finished (see pdl_wait in the kernels).
// cluster_z > 1 launches thread-block clusters of cluster_z CTAs along z (grid.z must be a multiple of it).
template <typename... KArgs, typename... Args>
cfi_status_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, int threads, size_t smem, int cluster_z,
                                cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2]{};
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = (unsigned)cluster_z;
    cfg.attrs = attr;
    cfg.numAttrs = cluster_z > 1 ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...) != cudaSuccess) {
        cudaGetLastError();
        return CFI_ERR_CUDA;
    }
    return CFI_OK;
}

template <typename... KArgs, typename... Args>
cfi_status_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, int threads, size_t smem, cudaStream_t st, Args... args) {
    return launch_pdl_cluster(kernel, grid, threads, smem, 1, st, args...);
}

template <typename VT, bool I16, int BT, int G>
cfi_status_t launch_splitk_g(const cfi_layer* l, const SplitkShape& s, const VT* x, VT* y, int batch,
                             cudaStream_t st) {
    if (s.xs == 8) {
        if (cfi_status_t e = set_smem<cfi_splitk_kernel<VT, I16, BT, G, 8>>(s.smem, l->device)) return e;
        return launch_pdl(cfi_splitk_kernel<VT, I16, BT, G, 8>, dim3(s.grid_x, s.grid_y), s.threads, s.smem, st, l->d, x, y, batch,
                          s.rows_per_group);
    }
    if (cfi_status_t e = set_smem<cfi_splitk_kernel<VT, I16, BT, G, 4>>(s.smem, l->device)) return e;
    return launch_pdl(cfi_splitk_kernel<VT, I16, BT, G, 4>, dim3(s.grid_x, s.grid_y), s.threads, s.smem, st, l->d, x, y, batch,
                      s.rows_per_group);
}

template <typename VT, bool I16, int BT>
cfi_status_t launch_splitk_i(const cfi_layer* l, const SplitkShape& s, const VT* x, VT* y, int batch, cudaStream_t st) {
    switch (s.g) {
        case 4: return launch_splitk_g<VT, I16, BT, 4>(l, s, x, y, batch, st);
        case 8: return launch_splitk_g<VT, I16, BT, 8>(l, s, x, y, batch, st);
        case 16: return launch_splitk_g<VT, I16, BT, 16>(l, s, x, y, batch, st);
        case 32: return launch_splitk_g<VT, I16, BT, 32>(l, s, x, y, batch, st);
    }
    return CFI_ERR_SHAPE;
}

template <typename VT, int BT>
cfi_status_t launch_splitk_bt(const cfi_layer* l, const SplitkShape& s, const VT* x, VT* y, int batch,
                              cudaStream_t st) {
    return l->d.idx16 ? launch_splitk_i<VT, true, BT>(l, s, x, y, batch, st) : launch_splitk_i<VT, false, BT>(l, s, x, y, batch, st);
}

template <typename VT>
cfi_status_t launch_splitk(const cfi_layer* l, const SplitkShape& s, const void* x, void* y, int batch,
                           cudaStream_t st) {
    if (!(l->layouts & CFI_LAYOUT_SMALL_BATCH)) return CFI_ERR_SHAPE;
    if (s.smem > (size_t)l->smem_optin || s.grid_y > 65535) return CFI_ERR_SHAPE;
    const VT* xx = static_cast<const VT*>(x);
    VT* yy = static_cast<VT*>(y);
    switch (s.bt) {
        case 1: return launch_splitk_bt<VT, 1>(l, s, xx, yy, batch, st);
        case 2: return launch_splitk_bt<VT, 2>(l, s, xx, yy, batch, st);
        case 4: return launch_splitk_bt<VT, 4>(l, s, xx, yy, batch, st);
        case 8: return launch_splitk_bt<VT, 8>(l, s, xx, yy, batch, st);
    }
    return CFI_ERR_SHAPE;
}

template <typename VT, int RPH>
cfi_status_t launch_batch_rph(const cfi_layer* l, const BatchShape& s, const VT* x, VT* y, int batch, cudaStream_t st) {
    if (cfi_status_t e = set_smem<cfi_batch_kernel<VT, kBatchTile, RPH>>(s.smem, l->device)) return e;
    return launch_pdl(cfi_batch_kernel<VT, kBatchTile, RPH>, dim3(s.grid_x, s.grid_y), s.threads, s.smem, st, l->d, x, y, batch);
}

template <typename VT>
cfi_status_t launch_batch(const cfi_layer* l, const BatchShape& s, const void* x, void* y, int batch,
                          cudaStream_t st) {
    if (!s.ok || s.grid_y > 65535) return CFI_ERR_SHAPE;
    const VT* xx = static_cast<const VT*>(x);
    VT* yy = static_cast<VT*>(y);
    switch (s.rph) {
        case 1: return launch_batch_rph<VT, 1>(l, s, xx, yy, batch, st);
        case 2: return launch_batch_rph<VT, 2>(l, s, xx, yy, batch, st);
        case 3: return launch_batch_rph<VT, 3>(l, s, xx, yy, batch, st);
        case 4: return launch_batch_rph<VT, 4>(l, s, xx, yy, batch, st);
        case 5: return launch_batch_rph<VT, 5>(l, s, xx, yy, batch, st);
        case 6: return launch_batch_rph<VT, 6>(l, s, xx, yy, batch, st);
        case 7: return launch_batch_rph<VT, 7>(l, s, xx, yy, batch, st);
        case 8: return launch_batch_rph<VT, 8>(l, s, xx, yy, batch, st);
    }
    return CFI_ERR_SHAPE;
}

template <typename VT>
cfi_status_t launch_simple(const cfi_layer* l, const void* x, void* y, int batch, cudaStream_t st) {
    if (!(l->layouts & CFI_LAYOUT_SMALL_BATCH)) return CFI_ERR_SHAPE;
    const int64_t total = (int64_t)batch * l->d.out;
    const int threads = 256;
    const int64_t blocks = (total + threads - 1) / threads;
    if (blocks > 0x7fffffffLL) return CFI_ERR_SHAPE;
    cfi_simple_kernel<VT><<<(unsigned)blocks, threads, 0, st>>>(l->d, static_cast<const VT*>(x), static_cast<VT*>(y),
                                                              batch);
    return cudaGetLastError() == cudaSuccess ? CFI_OK : CFI_ERR_CUDA;
}

// cuTensorMapEncodeTiled is a driver entry point; it is looked up once through the runtime so that the library
// does not link against the driver directly.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
    static std::atomic<void*> cached{nullptr};
    void* fn = cached.load(std::memory_order_acquire);
    if (!fn) {
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        cached.store(fn, std::memory_order_release);
    }
    return reinterpret_cast<EncodeTiledFn>(fn);
}

// Tensor map of a row-major bf16 or fp32 matrix [rows][cols] read in boxes of box_rows rows x 128 bytes of columns
// with the 128-byte swizzle; out-of-range elements read as zero.  Needs a 16-byte aligned base and row pitch.
bool encode_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, int elem_bytes, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn || rows == 0 || cols == 0 || ((cols * elem_bytes) & 15) || ((uintptr_t)base & 15)) return false;
    const cuuint64_t dims[2] = {cols, rows}, strides[1] = {cols * (uint64_t)elem_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)(128 / elem_bytes), (cuuint32_t)box_rows}, elem[2] = {1, 1};
    return fn(map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
              const_cast<void*>(base), dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kMaxSplit = kMaxClusterSplit;

// Time model of the split-TF32 kernel (fp32 layers on the tensor cores; measured): seconds per 32-column block of K by
// batch tile, a fixed part per wave of CTAs (prologue, pipeline fill, epilogue: CTAs are not persistent, so a second
// wave pays it again), the cluster reduction when K is split, and the launch itself.  The dense weight pieces
// (4 bytes per dense entry) have to come from HBM at least once per call.
constexpr double kSplitLaunch = 0.7e-6, kSplitWave = 4.2e-6, kSplitHbmBytesPerSecond = 5.5e12;
double split_seconds_per_block(int bt) { return bt >= 128 ? 0.51e-6 : bt >= 96 ? 0.40e-6 : 0.31e-6; }  // the issue of 4 + 4 MMAs and a commit
double split_seconds_reduce(int bt) { return 0.5e-6 + 0.95e-6 * bt / 128.0; }
int split_bt_index(int bt) {
    for (int i = 0; i < kSpNumTiles; ++i)
        if (kSpTiles[i] == bt) return i;
    return -1;
}

template <int BT>
int split_query_clusters(const cfi_layer* l, int split) {
    if (set_smem<cfi_dense_split_kernel<BT>>(sp_smem_bytes(BT), l->device) != CFI_OK) return 0;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(1, 1, (unsigned)split);
    cfg.blockDim = dim3(kSpThreads);
    cfg.dynamicSmemBytes = sp_smem_bytes(BT);
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 1, attr.val.clusterDim.y = 1, attr.val.clusterDim.z = (unsigned)split;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, cfi_dense_split_kernel<BT>, &cfg) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

// Clusters of `split` CTAs of the split-TF32 kernel that the device can hold at once; 0 if it cannot launch that
// cluster size (cached per device; -1 in the cache stands for 0).
int split_resident_clusters(const cfi_layer* l, int bt, int split) {
    static std::atomic<int> cache[kMaxDevices][kSpNumTiles][kMaxSplit + 1];
    if (split == 1) return std::max(1, l->sm_count);
    const int ti = split_bt_index(bt);
    if (l->device < 0 || l->device >= kMaxDevices || ti < 0) return 0;
    std::atomic<int>& c = cache[l->device][ti][split];
    int v = c.load(std::memory_order_acquire);
    if (v == 0) {
        switch (bt) {
            case 16: v = split_query_clusters<16>(l, split); break;
            case 32: v = split_query_clusters<32>(l, split); break;
            case 48: v = split_query_clusters<48>(l, split); break;
            case 64: v = split_query_clusters<64>(l, split); break;
            case 96: v = split_query_clusters<96>(l, split); break;
            default: v = split_query_clusters<128>(l, split); break;
        }
        if (v <= 0) v = -1;
        c.store(v, std::memory_order_release);
    }
    return v > 0 ? v : 0;
}

struct SplitShape {
    int bt;          // batch rows per tile: one of kSpTiles (the MMA's N is twice that)
    int split;       // CTAs per output tile (cluster size along z): 1 .. 8
    double seconds;  // modelled time of the launch
    bool ok;
};

// Batch tile and K split: a narrower batch tile costs less per K block, a wider one shares each weight box among more
// batch rows; splitting K over a cluster fills the SMs that the tiles alone would leave idle, as long as every CTA
// still gets a few K blocks.  force_bt / force_split (0 = free) pin one or both.
SplitShape split_shape(const cfi_layer* l, int batch, int force_bt = 0, int force_split = 0) {
    const int k_blocks = (l->d.in + kSpK - 1) / kSpK, tiles_m = (l->d.out + kSpM - 1) / kSpM;
    const double t_hbm = 4.0 * l->out_pad * (double)l->d.in / kSplitHbmBytesPerSecond;
    SplitShape best{128, 1, 0.0, false};
    for (int bt : kSpTiles) {
        if (force_bt && bt != force_bt) continue;
        const int64_t tiles_b = (batch + bt - 1) / bt;
        if (tiles_b > 65535) continue;
        const int64_t tiles = tiles_m * tiles_b;
        for (int split = 1; split <= kMaxSplit; ++split) {
            if (force_split ? split != force_split : (split > 1 && (k_blocks < 2 * split || tiles * split > 2 * (int64_t)l->sm_count))) continue;
            const int64_t resident = split_resident_clusters(l, bt, split);
            if (resident == 0) continue;
            const int64_t waves = (tiles + resident - 1) / resident;
            const double main = (double)waves * ((k_blocks + split - 1) / split) * split_seconds_per_block(bt);
            const double t = std::max(main, t_hbm) + (double)waves * (kSplitWave + (split > 1 ? split_seconds_reduce(bt) : 0.0)) + kSplitLaunch;
            if (!best.ok || t < best.seconds) best = SplitShape{bt, split, t, true};
        }
    }
    return best;
}

template <int BT>
cfi_status_t launch_dense_split_bt(const cfi_layer* l, int split, const void* x, void* y, int batch, cudaStream_t st) {
    const int grid_x = (l->d.out + kSpM - 1) / kSpM, grid_y = (batch + BT - 1) / BT;
    CUtensorMap map_x;  // x in boxes of BT rows x 32 columns
    if (!encode_map(&map_x, x, (uint64_t)batch, (uint64_t)l->d.in, 4, BT)) return CFI_ERR_SHAPE;
    if (cfi_status_t e = set_smem<cfi_dense_split_kernel<BT>>(sp_smem_bytes(BT), l->device)) return e;
    return launch_pdl_cluster(cfi_dense_split_kernel<BT>, dim3(grid_x, grid_y, split), kSpThreads, sp_smem_bytes(BT), split, st, l->d,
                              l->map_w, map_x, static_cast<float*>(y), batch);
}

cfi_status_t launch_dense_split(const cfi_layer* l, const void* x, void* y, int batch, cudaStream_t st, int force_bt = 0,
                                int force_split = 0) {
    if (force_bt && split_bt_index(force_bt) < 0) return CFI_ERR_SHAPE;
    if (force_split < 0 || force_split > kMaxSplit) return CFI_ERR_SHAPE;
    const SplitShape sh = split_shape(l, batch, force_bt, force_split);
    if (!sh.ok) return CFI_ERR_SHAPE;
    switch (sh.bt) {
        case 16: return launch_dense_split_bt<16>(l, sh.split, x, y, batch, st);
        case 32: return launch_dense_split_bt<32>(l, sh.split, x, y, batch, st);
        case 48: return launch_dense_split_bt<48>(l, sh.split, x, y, batch, st);
        case 64: return launch_dense_split_bt<64>(l, sh.split, x, y, batch, st);
        case 96: return launch_dense_split_bt<96>(l, sh.split, x, y, batch, st);
        default: return launch_dense_split_bt<128>(l, sh.split, x, y, batch, st);
    }
}

// bf16: with at least one 128 x 256 tile per SM the persistent kernel runs (measured: faster from about there
// on), else one 128 x 128 tile per CTA.
bool tc_bf16_persistent(const cfi_layer* l, int batch) {
    const int64_t n_tiles = (int64_t)((l->d.out + kTpN - 1) / kTpN) * ((batch + kTcM - 1) / kTcM);
    return n_tiles >= (int64_t)l->sm_count && n_tiles < (1ll << 31);
}

// Clusters of `split` CTAs of the one-tile bf16 kernel that the device can hold at once; 0 if it cannot launch that
// cluster size (cached per device; -1 in the cache stands for 0).  Both activations have the same footprint.
int tc_bf16_resident_clusters(const cfi_layer* l, int split) {
    static std::atomic<int> cache[64][kMaxSplit + 1];
    if (split == 1) return std::max(1, 2 * l->sm_count);
    if (l->device < 0 || l->device >= 64) return 0;
    std::atomic<int>& c = cache[l->device][split];
    int v = c.load(std::memory_order_acquire);
    if (v == 0) {
        v = -1;
        if (set_smem<cfi_dense_tc_kernel<CFI_ACT_GELU_ERF>>(kTcSmemBytes, l->device) == CFI_OK) {
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3(1, 1, (unsigned)split);
            cfg.blockDim = dim3(kTcThreads);
            cfg.dynamicSmemBytes = kTcSmemBytes;
            cudaLaunchAttribute attr{};
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = 1, attr.val.clusterDim.y = 1, attr.val.clusterDim.z = (unsigned)split;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, cfi_dense_tc_kernel<CFI_ACT_GELU_ERF>, &cfg) == cudaSuccess && n > 0) v = n;
            else cudaGetLastError();
        }
        c.store(v, std::memory_order_release);
    }
    return v > 0 ? v : 0;
}

// K split of the one-tile bf16 kernel: as for the split-TF32 kernel, a time model over the cluster sizes (seconds
// per 64-column block of K, a fixed part per wave of CTAs, the cluster reduction, the launch; measured).
int tc_bf16_split(const cfi_layer* l, int batch, double* seconds = nullptr) {
    const int64_t tiles = (int64_t)((batch + kTcM - 1) / kTcM) * ((l->d.out + kTcN - 1) / kTcN);
    const int k_blocks = (l->d.in + kTcK - 1) / kTcK;
    int best = 1;
    double best_t = 0.0;
    for (int split = 1; split <= kMaxSplit; ++split) {
        if (split > 1 && (k_blocks < 4 * split || tiles * split > 4 * (int64_t)l->sm_count)) break;
        const int64_t resident = tc_bf16_resident_clusters(l, split);
        if (resident == 0) continue;
        const int64_t waves = (tiles + resident - 1) / resident;
        const double t = (double)waves * (((k_blocks + split - 1) / split) * 0.27e-6 + 3.0e-6 + (split > 1 ? 1.0e-6 : 0.0)) + 0.7e-6;
        if (split == 1 || t < best_t) best = split, best_t = t;
    }
    if (seconds) *seconds = best_t;
    return best;
}

// tile / cluster: 0 = chosen here.  fp32 layers: tile = batch rows per tile (16, 32, 64, 128); bf16 layers: tile = outputs
// per tile, 128 (one tile per CTA, K may be split over `cluster` CTAs) or 256 (persistent kernel, no split).
cfi_status_t launch_dense_tc(const cfi_layer* l, const void* x, void* y, int batch, cudaStream_t st, int tile = 0,
                             int cluster = 0) {
    if (!l->tc_ok) return CFI_ERR_SHAPE;
    if (l->dtype != CFI_BF16) return launch_dense_split(l, x, y, batch, st, tile, cluster);
    if ((tile != 0 && tile != kTcN && tile != kTpN) || cluster < 0 || cluster > kMaxSplit || (tile == kTpN && cluster > 1))
        return CFI_ERR_SHAPE;
    const int grid_x = (l->d.out + kTcN - 1) / kTcN, grid_y = (batch + kTcM - 1) / kTcM;
    if (grid_y > 65535) return CFI_ERR_SHAPE;
    CUtensorMap map_x;
    if (!encode_map(&map_x, x, (uint64_t)batch, (uint64_t)l->d.in, 2, kTcM)) return CFI_ERR_SHAPE;
    // A tile or more per SM: one persistent CTA per SM with 128 x 256 tiles that overlaps each tile's epilogue with
    // the next tile's MMAs.
    const int wide_x = (l->d.out + kTpN - 1) / kTpN;
    const int64_t n_tiles = (int64_t)wide_x * grid_y;
    if (tile == kTpN || (tile == 0 && cluster == 0 && tc_bf16_persistent(l, batch))) {
        if (n_tiles >= (1ll << 31)) return CFI_ERR_SHAPE;
        const int ctas = (int)std::min<int64_t>(l->sm_count, n_tiles);
        CUtensorMap map_y;  // y leaves through TMA stores of 128-row x 64-column boxes
        if (!encode_map(&map_y, y, (uint64_t)batch, (uint64_t)l->d.out, 2, kTcM)) return CFI_ERR_SHAPE;
        if (l->d.act == CFI_ACT_GELU_ERF) {
            if (cfi_status_t e = set_smem<cfi_dense_tc_persistent_kernel<CFI_ACT_GELU_ERF>>(kTpSmemBytes, l->device)) return e;
            return launch_pdl(cfi_dense_tc_persistent_kernel<CFI_ACT_GELU_ERF>, dim3(ctas), kTpThreads, kTpSmemBytes, st, l->d,
                              map_x, l->map_w_wide, map_y, batch, wide_x, (int)n_tiles);
        }
        if (cfi_status_t e = set_smem<cfi_dense_tc_persistent_kernel<CFI_ACT_NONE>>(kTpSmemBytes, l->device)) return e;
        return launch_pdl(cfi_dense_tc_persistent_kernel<CFI_ACT_NONE>, dim3(ctas), kTpThreads, kTpSmemBytes, st, l->d, map_x,
                          l->map_w_wide, map_y, batch, wide_x, (int)n_tiles);
    }
    const int split = cluster ? cluster : tc_bf16_split(l, batch);
    if (split > 1 && tc_bf16_resident_clusters(l, split) == 0) return CFI_ERR_SHAPE;
    if (l->d.act == CFI_ACT_GELU_ERF) {
        if (cfi_status_t e = set_smem<cfi_dense_tc_kernel<CFI_ACT_GELU_ERF>>(kTcSmemBytes, l->device)) return e;
        return launch_pdl_cluster(cfi_dense_tc_kernel<CFI_ACT_GELU_ERF>, dim3(grid_x, grid_y, split), kTcThreads, kTcSmemBytes,
                                  split, st, l->d, map_x, l->map_w, static_cast<__nv_bfloat16*>(y), batch);
    }
    if (cfi_status_t e = set_smem<cfi_dense_tc_kernel<CFI_ACT_NONE>>(kTcSmemBytes, l->device)) return e;
    return launch_pdl_cluster(cfi_dense_tc_kernel<CFI_ACT_NONE>, dim3(grid_x, grid_y, split), kTcThreads, kTcSmemBytes, split, st,
                              l->d, map_x, l->map_w, static_cast<__nv_bfloat16*>(y), batch);
}

// Clusters of `split` CTAs of the slab kernel with `smem` bytes of shared memory each that the device holds at once
// (cached per device, storage type, cluster size and 8 KB step of shared memory; 0 if unknown).
int slab_resident_clusters(const cfi_layer* l, int split, size_t smem) {
    static std::atomic<int> cache[kMaxDevices][2][4][32];
    const int bf = l->dtype == CFI_BF16 ? 1 : 0, ls = split >= 8 ? 3 : split >= 4 ? 2 : split >= 2 ? 1 : 0;
    const int step = (int)std::min<size_t>(31, smem >> 13);
    if (l->device < 0 || l->device >= kMaxDevices) return 0;
    std::atomic<int>& c = cache[l->device][bf][ls][step];
    int v = c.load(std::memory_order_acquire);
    if (v == 0) {
        v = -1;
        const size_t bytes = ((size_t)step + 1) << 13;  // the step's upper end
        const bool set = bf ? set_smem<cfi_slab_kernel<__nv_bfloat16>>(bytes, l->device) == CFI_OK
                            : set_smem<cfi_slab_kernel<float>>(bytes, l->device) == CFI_OK;
        if (set) {
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3((unsigned)split, 1, 1);
            cfg.blockDim = dim3(kSlabThreads);
            cfg.dynamicSmemBytes = bytes;
            cudaLaunchAttribute attr{};
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = (unsigned)split, attr.val.clusterDim.y = 1, attr.val.clusterDim.z = 1;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            int n = 0;
            const cudaError_t e = bf ? cudaOccupancyMaxActiveClusters(&n, cfi_slab_kernel<__nv_bfloat16>, &cfg)
                                     : cudaOccupancyMaxActiveClusters(&n, cfi_slab_kernel<float>, &cfg);
            if (e == cudaSuccess && n > 0) v = n;
            else cudaGetLastError();
        }
        c.store(v, std::memory_order_release);
    }
    return v > 0 ? v : 0;
}

// Launch shape of the slab kernel: S CTAs of a cluster share a group of rows and divide the column slabs (the fewest
// for which a CTA's columns of a 16-row batch tile take at most 96 KB, so that two CTAs fit an SM), and the rows are
// divided into as many groups as the device holds clusters at once: one wave.
struct SlabShape { int split, groups, rows_pc, tiles, ncols_max; size_t smem; bool ok; };

SlabShape slab_shape(const cfi_layer* l, int batch) {
    SlabShape s{};
    s.ok = false;
    if (!(l->layouts & CFI_LAYOUT_GATHER) || l->d.out < 1 || batch < 1) return s;
    s.tiles = (batch + kSlabBT - 1) / kSlabBT;
    if (s.tiles > 65535) return s;
    for (int split = 1; split <= kMaxClusterSplit; split <<= 1) {
        const int nsl_max = (l->d.n_slabs + split - 1) / split, ncols_max = nsl_max * l->d.cs;
        const size_t xbytes = (size_t)(ncols_max + 1) * kSlabBT * 4;
        if (xbytes > 96 * 1024 && split < kMaxClusterSplit) continue;
        s.split = split, s.ncols_max = ncols_max;
        auto with_groups = [&](int64_t want) {
            const int groups = (int)std::max<int64_t>(1, std::min<int64_t>(want, (l->d.out + kSlabWarps - 1) / kSlabWarps));
            s.rows_pc = (l->d.out + groups - 1) / groups;
            s.groups = (l->d.out + s.rows_pc - 1) / s.rows_pc;
            s.smem = xbytes + (size_t)s.rows_pc * kSlabBT * 4 + (size_t)s.rows_pc * (nsl_max + 2) * 4;
        };
        with_groups((2 * (int64_t)l->sm_count) / ((int64_t)split * s.tiles));
        if (s.smem <= (size_t)l->smem_optin) {
            const int resident = slab_resident_clusters(l, split, s.smem);
            if (resident > 0 && (int64_t)s.groups * s.tiles > resident) with_groups(resident / s.tiles);
        }
        s.ok = s.smem <= (size_t)l->smem_optin && s.groups <= 65535;
        return s;
    }
    return s;
}

template <typename VT>
cfi_status_t launch_slab(const cfi_layer* l, const void* x, void* y, int batch, cudaStream_t st) {
    const SlabShape s = slab_shape(l, batch);
    if (!s.ok) return CFI_ERR_SHAPE;
    if (cfi_status_t e = set_smem<cfi_slab_kernel<VT>>(s.smem, l->device)) return e;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)s.split, (unsigned)s.groups, (unsigned)s.tiles);
    cfg.blockDim = dim3(kSlabThreads);
    cfg.dynamicSmemBytes = s.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2]{};
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)s.split;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = s.split > 1 ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, cfi_slab_kernel<VT>, l->d, static_cast<const VT*>(x), static_cast<VT*>(y), batch, s.rows_pc,
                           s.ncols_max) != cudaSuccess) {
        cudaGetLastError();
        return CFI_ERR_CUDA;
    }
    return CFI_OK;
}

// Rate of the gather kernel's arithmetic, used to choose between it and the split-TF32 dense kernel (measured).
constexpr double kGatherTflops = 12.5;

// The split-k kernel keeps at least one whole row of x (+ one zero element) in shared memory.
bool splitk_fits(const cfi_layer* l, int batch) {
    return (l->layouts & CFI_LAYOUT_SMALL_BATCH) && splitk_shape(l, batch).smem <= (size_t)l->smem_optin;
}

// What remains when the preferred kernel cannot hold its tile: the gather kernel (column slabs), else one thread per output.
int fallback_variant(const cfi_layer* l, int batch) {
    if (batch_shape(l, batch).ok) return CFI_VARIANT_BATCH;
    if (splitk_fits(l, batch)) return CFI_VARIANT_SPLITK;
    if (l->tc_ok && !(l->layouts & CFI_LAYOUT_SMALL_BATCH)) return CFI_VARIANT_DENSE_TC;
    return CFI_VARIANT_SIMPLE;
}

// Time model of the slab kernel (measured, fp32): a fixed part (cluster launch, row table, staging of x, cluster
// reduction) and the entries of all batch tiles at the rate the gathers sustain.
double slab_seconds(const cfi_layer* l, int batch) {
    return 10.8e-6 + 4.4e-12 * (double)l->d.n_active * l->d.k * ((batch + kSlabBT - 1) / kSlabBT);
}

int choose_variant(const cfi_layer* l, int batch) {
    // A layer built without the small-batch layout runs every batch size on what it has.
    if (!(l->layouts & CFI_LAYOUT_SMALL_BATCH) && batch <= 24)
        return l->tc_ok && (batch > 4 || !batch_shape(l, batch).ok) ? CFI_VARIANT_DENSE_TC : fallback_variant(l, batch);
    // Up to three batch tiles of 8 the split-k kernel (weights re-read from L2 per tile) beats the 64-wide tiles of
    // the batch kernel, which would be mostly empty.
    if (batch <= 24) {
        // Two or three passes of the split-k kernel over a large fp32 layer can take longer than the tensor-core
        // variant does for any batch up to 128 (measured 4096 x 4096 at 80 %, batch 16: 31 against 25 us; 3072 -> 768:
        // 22 against 11 us).  A pass of eight batch rows costs about 2.3 us plus the larger of staging x (90 ns per KB
        // of the 8-row tile, every CTA stages all of it) and the weights (176 G entries per second).
        if (batch > 8) {
            constexpr double kNever = 1e30;
            const double t_stage = (double)l->d.in * 8 * 4 / 1024.0 * 90e-9, t_fma = (double)l->d.n_active * l->d.k / 176e9;
            const double t_splitk = splitk_fits(l, batch) ? ((batch + 7) / 8) * (2.3e-6 + std::max(t_stage, t_fma)) : kNever;
            double t_dense = kNever;
            if (l->tc_ok && l->dtype == CFI_F32) t_dense = split_shape(l, batch).seconds;
            else if (l->tc_ok) tc_bf16_split(l, batch, &t_dense);
            // Very sparse fp32 layers: the condensed arrays are far smaller than the dense copy, and the slab kernel
            // reads only them.
            if (l->dtype == CFI_F32 && slab_seconds(l, batch) < std::min(t_dense, t_splitk) && slab_shape(l, batch).ok)
                return CFI_VARIANT_SLAB;
            if (t_dense < t_splitk) return CFI_VARIANT_DENSE_TC;
        }
        return splitk_fits(l, batch) ? CFI_VARIANT_SPLITK : fallback_variant(l, batch);
    }
    // bf16 above 24 rows: the dense contraction on the tensor cores beats the gather kernel even at 99 % sparsity
    // (10 TFLOP/s effective for the gather against several hundred dense), also with a partly empty 128-row tile
    // now that K can be split over a cluster (3072 -> 768 at batch 64: 8.5 against 33 us).
    if (l->tc_ok && l->dtype == CFI_BF16) return CFI_VARIANT_DENSE_TC;
    if (l->tc_ok && l->dtype == CFI_F32) {
        // fp32: the split-TF32 kernel takes a fixed time per 32-column block of K and tile (it is bound by the
        // number of MMA instructions), whatever the fill of its 128-row batch tile, and can split K over a cluster
        // when the tiles are few; the gather kernel's time is its FMAs at the rate it sustains plus the re-staging
        // of x by every row tile.  Constants fitted to measurements.
        const BatchShape bs = batch_shape(l, batch);
        if (!bs.ok) return CFI_VARIANT_DENSE_TC;
        const double t_dense = split_shape(l, batch).seconds;
        const double staging = (double)bs.grid_y * kBatchTile * l->d.in * 4.0 * bs.grid_x;
        // Arithmetic and the re-staging of x overlap about half of the shorter of the two.
        const double t_fma = 2.0 * batch * (double)l->d.n_active * l->d.k / (kGatherTflops * 1e12), t_stage = staging / 3.7e12;
        const double t_gather = t_fma + t_stage - 0.5 * std::min(t_fma, t_stage) + 5e-6;
        if (batch <= 64 && slab_seconds(l, batch) < std::min(t_dense, t_gather) && slab_shape(l, batch).ok) return CFI_VARIANT_SLAB;
        if (t_dense < t_gather) return CFI_VARIANT_DENSE_TC;
    }
    if (batch <= 64 && l->dtype == CFI_F32 && !l->tc_ok && slab_shape(l, batch).ok) {
        // Without a dense copy: the slab kernel against the gather kernel's 64-wide, partly empty batch tiles.
        const BatchShape bs = batch_shape(l, batch);
        if (!bs.ok || slab_seconds(l, batch) < 2.0 * batch * (double)l->d.n_active * l->d.k / (kGatherTflops * 1e12) * (64.0 / std::min(batch, 64)) + 8e-6)
            return CFI_VARIANT_SLAB;
    }
    return fallback_variant(l, batch);
}

// ------------------------------------------------------------------------------------------------
// host: construction
// ------------------------------------------------------------------------------------------------
uint16_t bf16_bits_rne(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return (uint16_t)((u >> 16) | 0x0040u);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

float bf16_widen(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}

struct DeviceGuard {
    int prev = -1;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) cudaSetDevice(dev);
        else prev = -1;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

template <typename T>
cfi_status_t upload(cfi_layer* l, const std::vector<T>& host, const T** dev) {
    void* p = nullptr;
    const size_t bytes = std::max<size_t>(host.size() * sizeof(T), 16);
    if (cudaMalloc(&p, bytes) != cudaSuccess) {
        cudaGetLastError();
        return CFI_ERR_ALLOC;
    }
    l->allocs.push_back(p);
    l->device_bytes += (int64_t)bytes;
    if (!host.empty() && cudaMemcpy(p, host.data(), host.size() * sizeof(T), cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError();
        return CFI_ERR_CUDA;
    }
    *dev = static_cast<const T*>(p);
    return CFI_OK;
}

// Order of a row's entries in the small-batch layout.  The `lanes` lanes that share a row read vector
// v = lane + lanes * t of the row and gather its element e in the same instruction, so the entries at
// positions vec * (lane + lanes * t) + e, lane = 0..lanes-1, hit shared memory together.  Entries are dealt
// to these sets so that a set's columns fall into different banks (column mod 32 for one batch row) as far
// as the row allows, lanes ascending with the bank so that aligned sub-groups differ in the low bits too.
// cols: the row's k columns; place[j] receives the position (< kp) of entry j; pad positions stay free.
void order_for_banks(const int32_t* cols, int k, int kp, int vec, int lanes, int32_t* place) {
    std::vector<int32_t> by_bank[32];
    for (int j = 0; j < k; ++j) by_bank[cols[j] & 31].push_back(j);
    const int nvec = kp / vec;
    int left = k;
    int order[32], chosen[32];
    for (int t = 0; t * lanes < nvec && left > 0; ++t) {
        const int width = std::min(lanes, nvec - t * lanes);  // lanes that have a vector in this round
        for (int e = 0; e < vec && left > 0; ++e) {
            // Fullest banks first; one entry per bank while enough banks are non-empty.
            std::iota(order, order + 32, 0);
            std::stable_sort(order, order + 32, [&](int a, int b) { return by_bank[a].size() > by_bank[b].size(); });
            const int quota = std::min(width, left);  // sets are filled in order; pads collect at the row's end
            int n_chosen = 0;
            for (int pass = 0; n_chosen < quota; ++pass)
                for (int q = 0; q < 32 && n_chosen < quota; ++q)
                    if ((int)by_bank[order[q]].size() > pass) chosen[n_chosen++] = order[q];
            std::sort(chosen, chosen + n_chosen);
            for (int i = 0; i < n_chosen; ++i) {
                const int j = by_bank[chosen[i]].back();
                by_bank[chosen[i]].pop_back();
                place[j] = vec * (i + lanes * t) + e;
                --left;
            }
        }
    }
}

void free_layer(cfi_layer* l) {
    for (void* p : l->allocs) cudaFree(p);
    if (l->stage_x) cudaFree(l->stage_x);
    if (l->stage_y) cudaFree(l->stage_y);
    delete l;
}

// Small-batch ("split-k") layout: values and indices padded to whole 16-byte vectors, entries ordered for the banks.
cfi_status_t build_small(cfi_layer* l) {
    const int32_t k = l->d.k, n_active = l->d.n_active, in_features = l->d.in, out_features = l->d.out;
    const int dtype = l->dtype;
    DevLayer& d = l->d;
    const std::vector<float>& v_sorted = l->h_values;
    const std::vector<int32_t>&c_sorted = l->h_cols, &active_rows = l->h_rows, &slot = l->h_slot;
    cfi_status_t st = CFI_OK;
    const int64_t before = l->device_bytes;
    (void)k, (void)n_active, (void)in_features, (void)out_features, (void)dtype, (void)d, (void)v_sorted, (void)c_sorted,
        (void)active_rows, (void)slot;
    // ---- small-batch layout
    const int vec = vec_of(dtype, d.idx16 != 0);
    d.kp = ((k + vec - 1) / vec) * vec;
    std::vector<int32_t> place((size_t)std::max(d.kp, 1));  // position in the padded row of sorted entry j
    const int lanes = splitk_lanes_per_row(std::max(1, d.kp / vec), splitk_units_in_flight(dtype == CFI_F32, d.idx16 != 0));
    std::vector<int32_t> idx_p((size_t)n_active * d.kp, in_features);
    if (dtype == CFI_F32) {
        std::vector<float> val_p((size_t)n_active * d.kp, 0.0f);
        for (int32_t r = 0; r < n_active; ++r) {
            order_for_banks(&c_sorted[(size_t)r * k], k, d.kp, vec, lanes, place.data());
            for (int32_t j = 0; j < k; ++j) {
                val_p[(size_t)r * d.kp + place[j]] = v_sorted[(size_t)r * k + j];
                idx_p[(size_t)r * d.kp + place[j]] = c_sorted[(size_t)r * k + j];
            }
        }
        const float* p = nullptr;
        st = upload(l, val_p, &p);
        d.values = p;
    } else {
        std::vector<uint16_t> val_p((size_t)n_active * d.kp, (uint16_t)0);
        for (int32_t r = 0; r < n_active; ++r) {
            order_for_banks(&c_sorted[(size_t)r * k], k, d.kp, vec, lanes, place.data());
            for (int32_t j = 0; j < k; ++j) {
                val_p[(size_t)r * d.kp + place[j]] = bf16_bits_rne(v_sorted[(size_t)r * k + j]);
                idx_p[(size_t)r * d.kp + place[j]] = c_sorted[(size_t)r * k + j];
            }
        }
        const uint16_t* p = nullptr;
        st = upload(l, val_p, &p);
        d.values = p;
    }
    if (st == CFI_OK) {
        if (d.idx16) {
            std::vector<uint16_t> idx16(idx_p.begin(), idx_p.end());
            const uint16_t* p = nullptr;
            st = upload(l, idx16, &p);
            d.indices = p;
        } else {
            const int32_t* p = nullptr;
            st = upload(l, idx_p, &p);
            d.indices = p;
        }
    }

    if (st == CFI_OK) l->layouts |= CFI_LAYOUT_SMALL_BATCH;
    l->bytes_small += l->device_bytes - before;
    return st;
}

// Large-batch gather layout: column slabs, 32-byte quads, per-row slab offsets.
cfi_status_t build_gather(cfi_layer* l) {
    const int32_t k = l->d.k, n_active = l->d.n_active, in_features = l->d.in, out_features = l->d.out;
    const int dtype = l->dtype;
    DevLayer& d = l->d;
    const std::vector<float>& v_sorted = l->h_values;
    const std::vector<int32_t>&c_sorted = l->h_cols, &active_rows = l->h_rows, &slot = l->h_slot;
    cfi_status_t st = CFI_OK;
    const int64_t before = l->device_bytes;
    (void)k, (void)n_active, (void)in_features, (void)out_features, (void)dtype, (void)d, (void)v_sorted, (void)c_sorted,
        (void)active_rows, (void)slot;
    // ---- large-batch layout: the fewest slabs (at least two when there is enough to pipeline) for which
    // two x buffers, the tile metadata and the per-warp weight buffers of the largest tile fit.
    const int es = dtype == CFI_BF16 ? 2 : 4;
    std::vector<int32_t> seg;
    for (int n_slabs = in_features >= 128 ? 2 : 1;; ++n_slabs) {
        d.cs = std::max(8, (((in_features + n_slabs - 1) / n_slabs) + 7) & ~7);
        d.n_slabs = std::max(1, (in_features + d.cs - 1) / d.cs);
        seg.assign((size_t)n_active * (d.n_slabs + 1), 0);
        int max_row_quads = 1, maxq = 1;
        for (int32_t r = 0; r < n_active; ++r) {
            int q = 0, j = 0;
            for (int s = 0; s < d.n_slabs; ++s) {
                seg[(size_t)r * (d.n_slabs + 1) + s] = q;
                int cnt = 0;
                while (j < k && c_sorted[(size_t)r * k + j] < (s + 1) * d.cs) ++j, ++cnt;
                q += (cnt + 3) / 4;
                maxq = std::max(maxq, (cnt + 3) / 4);
            }
            seg[(size_t)r * (d.n_slabs + 1) + d.n_slabs] = q;
            max_row_quads = std::max(max_row_quads, q);
        }
        d.stride_q = max_row_quads;
        d.maxq = maxq;
        const BatchSmem m = batch_smem_layout(d.cs, d.n_slabs, d.maxq, es, kBatchTile, 128, 8);
        if (m.total <= (size_t)kBatchSmemBudget || d.cs <= 8) break;
    }
    struct Quad { float w[4]; int32_t c[4]; };
    std::vector<Quad> quads((size_t)n_active * d.stride_q);
    for (auto& q : quads)
        for (int e = 0; e < 4; ++e) q.w[e] = 0.0f, q.c[e] = d.cs * kBatchTile * es;
    for (int32_t r = 0; r < n_active; ++r) {
        int j = 0;
        for (int s = 0; s < d.n_slabs; ++s) {
            size_t w = (size_t)seg[(size_t)r * (d.n_slabs + 1) + s] * 4;
            while (j < k && c_sorted[(size_t)r * k + j] < (s + 1) * d.cs) {
                Quad& q = quads[(size_t)r * d.stride_q + w / 4];
                q.w[w % 4] = v_sorted[(size_t)r * k + j];
                const int col = c_sorted[(size_t)r * k + j] - s * d.cs;
                q.c[w % 4] = col * kBatchTile * es + ((col >> 2) & (kBatchTile / 4 - 1)) * 4 * es;
                ++w, ++j;
            }
        }
    }
    const Quad* quads_dev = nullptr;
    if (st == CFI_OK) st = upload(l, quads, &quads_dev);
    d.wq_b = quads_dev;
    // The kernel looks the quad offsets up by output row: ablated rows get an all-zero line.
    std::vector<int32_t> seg_o((size_t)out_features * (d.n_slabs + 1), 0);
    for (int32_t o = 0; o < out_features; ++o)
        if (slot[o] >= 0)
            std::copy(seg.begin() + (size_t)slot[o] * (d.n_slabs + 1), seg.begin() + (size_t)(slot[o] + 1) * (d.n_slabs + 1),
                      seg_o.begin() + (size_t)o * (d.n_slabs + 1));
    if (st == CFI_OK) st = upload(l, seg_o, &d.seg);

    if (st == CFI_OK) l->layouts |= CFI_LAYOUT_GATHER;
    l->bytes_gather += l->device_bytes - before;
    return st;
}

// Dense copy for the tensor-core variant; leaves tc_ok false where the shapes cannot be addressed.
cfi_status_t build_dense(cfi_layer* l) {
    const int32_t k = l->d.k, n_active = l->d.n_active, in_features = l->d.in, out_features = l->d.out;
    const int dtype = l->dtype;
    DevLayer& d = l->d;
    const std::vector<float>& v_sorted = l->h_values;
    const std::vector<int32_t>&c_sorted = l->h_cols, &active_rows = l->h_rows, &slot = l->h_slot;
    cfi_status_t st = CFI_OK;
    const int64_t before = l->device_bytes;
    (void)k, (void)n_active, (void)in_features, (void)out_features, (void)dtype, (void)d, (void)v_sorted, (void)c_sorted,
        (void)active_rows, (void)slot;
    // ---- dense copy for the tensor-core variant (zero rows for ablated and padding rows), in the layer's dtype.
    // A column kept twice in one row cannot be one dense entry, so such layers go without.
    {
        const int eb = dtype == CFI_BF16 ? 2 : 4, tile_n = 128;
        bool usable = out_features > 0 && in_features * eb >= 16 && ((in_features * eb) & 15) == 0 &&
                      ((out_features * eb) & 15) == 0 && (size_t)out_features * in_features * eb <= ((size_t)1 << 30);
        for (int32_t r = 0; usable && r < n_active; ++r)
            for (int32_t j = 1; j < k; ++j) usable = usable && c_sorted[(size_t)r * k + j] != c_sorted[(size_t)r * k + j - 1];
        if (usable) {
            l->out_pad = ((out_features + tile_n - 1) / tile_n) * tile_n;
            const void* wd_dev = nullptr;
            if (dtype == CFI_BF16) {
                std::vector<uint16_t> wd((size_t)l->out_pad * in_features, (uint16_t)0);
                for (int32_t r = 0; r < n_active; ++r)
                    for (int32_t j = 0; j < k; ++j)
                        wd[(size_t)active_rows[r] * in_features + c_sorted[(size_t)r * k + j]] =
                            bf16_bits_rne(v_sorted[(size_t)r * k + j]);
                const uint16_t* p = nullptr;
                if (st == CFI_OK) st = upload(l, wd, &p);
                wd_dev = p;
            } else {
                std::vector<float> wd((size_t)l->out_pad * in_features, 0.0f);
                for (int32_t r = 0; r < n_active; ++r)
                    for (int32_t j = 0; j < k; ++j)
                        wd[(size_t)active_rows[r] * in_features + c_sorted[(size_t)r * k + j]] = v_sorted[(size_t)r * k + j];
                const float* p = nullptr;
                if (st == CFI_OK) st = upload(l, wd, &p);
                wd_dev = p;
            }
            l->w_dense = wd_dev;
            // Boxes of 128 rows x 128 bytes for the one-tile kernels; for bf16 layers also 256-row boxes for the
            // persistent kernel's wide tiles.
            l->tc_ok = st == CFI_OK && encode_map(&l->map_w, wd_dev, (uint64_t)l->out_pad, (uint64_t)in_features, eb, kTcN);
            if (l->tc_ok && dtype == CFI_BF16)
                l->tc_ok = encode_map(&l->map_w_wide, wd_dev, (uint64_t)l->out_pad, (uint64_t)in_features, 2, kTpN);
        }
    }

    if (st == CFI_OK && l->tc_ok) l->layouts |= CFI_LAYOUT_DENSE;
    l->bytes_dense += l->device_bytes - before;
    return st;
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------------------------
extern "C" cfi_status_t cfi_create(const float* values, const int32_t* indices, const int32_t* active_rows,
                                   const float* bias, int32_t n_active, int32_t k, int32_t in_features,
                                   int32_t out_features, cfi_dtype_t dtype, cfi_act_t act, cfi_layer_t** layer) {
    return cfi_create_layouts(values, indices, active_rows, bias, n_active, k, in_features, out_features, dtype, act,
                              CFI_LAYOUT_ALL, layer);
}

extern "C" cfi_status_t cfi_create_layouts(const float* values, const int32_t* indices, const int32_t* active_rows,
                                           const float* bias, int32_t n_active, int32_t k, int32_t in_features,
                                           int32_t out_features, cfi_dtype_t dtype, cfi_act_t act, int32_t layouts,
                                           cfi_layer_t** layer) {
    if (!layer) return CFI_ERR_NULL;
    *layer = nullptr;
    if (layouts <= 0 || (layouts & ~CFI_LAYOUT_ALL)) return CFI_ERR_DTYPE;
    if (dtype != CFI_F32 && dtype != CFI_BF16) return CFI_ERR_DTYPE;
    if (act != CFI_ACT_NONE && act != CFI_ACT_GELU_ERF) return CFI_ERR_DTYPE;
    if (n_active < 0 || k < 0 || in_features < 0 || out_features < 0) return CFI_ERR_SHAPE;
    if (n_active > out_features || k > in_features || in_features > (1 << 20)) return CFI_ERR_SHAPE;
    if (n_active > 0 && k < 1) return CFI_ERR_SHAPE;
    if (n_active > 0 && (!values || !indices || !active_rows)) return CFI_ERR_NULL;
    const size_t nnz = (size_t)n_active * (size_t)k;
    for (size_t i = 0; i < nnz; ++i)
        if (indices[i] < 0 || indices[i] >= in_features) return CFI_ERR_INDEX_RANGE;

    std::vector<int32_t> slot((size_t)out_features, -1);
    for (int32_t r = 0; r < n_active; ++r) {
        const int32_t o = active_rows[r];
        if (o < 0 || o >= out_features || slot[o] != -1) return CFI_ERR_INDEX_RANGE;
        slot[o] = r;
    }
    bool identity_rows = n_active == out_features;
    for (int32_t r = 0; identity_rows && r < n_active; ++r) identity_rows = active_rows[r] == r;

    cfi_layer* l = new (std::nothrow) cfi_layer();
    if (!l) return CFI_ERR_ALLOC;
    cudaDeviceProp prop{};
    if (cudaGetDevice(&l->device) != cudaSuccess || cudaGetDeviceProperties(&prop, l->device) != cudaSuccess) {
        cudaGetLastError();
        delete l;
        return CFI_ERR_CUDA;
    }
    l->sm_count = prop.multiProcessorCount;
    l->smem_optin = (int)prop.sharedMemPerBlockOptin;
    l->dtype = dtype;
    DevLayer& d = l->d;
    d.in = in_features, d.out = out_features, d.n_active = n_active, d.k = k, d.act = act;
    d.identity_rows = identity_rows ? 1 : 0;

    try {
        // Each row sorted by column (stable, so repeated columns keep the caller's order).
        std::vector<int32_t> order((size_t)std::max(k, 1));
        l->h_values.resize(nnz);
        l->h_cols.resize(nnz);
        l->h_rows.assign(active_rows, active_rows + n_active);
        l->h_slot = slot;
        for (int32_t r = 0; r < n_active; ++r) {
            const size_t off = (size_t)r * k;
            std::iota(order.begin(), order.begin() + k, 0);
            std::stable_sort(order.begin(), order.begin() + k,
                             [&](int32_t a, int32_t b) { return indices[off + a] < indices[off + b]; });
            for (int32_t j = 0; j < k; ++j) {
                float w = values[off + order[j]];
                if (dtype == CFI_BF16) w = bf16_widen(bf16_bits_rne(w));
                l->h_values[off + j] = w;
                l->h_cols[off + j] = indices[off + order[j]];
            }
        }
        d.idx16 = use_idx16(in_features, (int64_t)nnz) ? 1 : 0;
        const int vec = vec_of(dtype, d.idx16 != 0);
        d.kp = ((k + vec - 1) / vec) * vec;
        cfi_status_t st = CFI_OK;
        if (st == CFI_OK && (layouts & CFI_LAYOUT_SMALL_BATCH)) st = build_small(l);
        if (st == CFI_OK && (layouts & CFI_LAYOUT_GATHER)) st = build_gather(l);
        if (st == CFI_OK && (layouts & CFI_LAYOUT_DENSE)) st = build_dense(l);
        if (st == CFI_OK && l->layouts == 0) st = CFI_ERR_SHAPE;  // only the dense layout was asked for and it cannot be built
        std::vector<float> bias_h((size_t)out_features, 0.0f);
        if (bias) std::copy(bias, bias + out_features, bias_h.begin());
        if (st == CFI_OK) st = upload(l, bias_h, &d.bias);
        if (st == CFI_OK) st = upload(l, slot, &d.slot);
        std::vector<int32_t> zero(4, 0);
        const int32_t* status = nullptr;
        if (st == CFI_OK) st = upload(l, zero, &status);
        d.status = const_cast<int32_t*>(status);
        if (st != CFI_OK) {
            free_layer(l);
            return st;
        }
    } catch (const std::bad_alloc&) {
        free_layer(l);
        return CFI_ERR_ALLOC;
    }
    *layer = l;
    return CFI_OK;
}

extern "C" cfi_status_t cfi_layer_add_layouts(cfi_layer_t* layer, int32_t layouts) {
    if (!layer) return CFI_ERR_NULL;
    if (layouts <= 0 || (layouts & ~CFI_LAYOUT_ALL)) return CFI_ERR_DTYPE;
    DeviceGuard g(layer->device);
    const int missing = layouts & ~layer->layouts;
    cfi_status_t st = CFI_OK;
    try {
        if (st == CFI_OK && (missing & CFI_LAYOUT_SMALL_BATCH)) st = build_small(layer);
        if (st == CFI_OK && (missing & CFI_LAYOUT_GATHER)) st = build_gather(layer);
        if (st == CFI_OK && (missing & CFI_LAYOUT_DENSE) && !layer->w_dense) st = build_dense(layer);
    } catch (const std::bad_alloc&) {
        return CFI_ERR_ALLOC;
    }
    return st;
}

extern "C" cfi_status_t cfi_destroy(cfi_layer_t* layer) {
    if (!layer) return CFI_OK;
    DeviceGuard g(layer->device);
    free_layer(layer);
    return CFI_OK;
}

extern "C" cfi_status_t cfi_choose_variant(const cfi_layer_t* layer, int32_t batch, int32_t* variant) {
    if (!layer || !variant) return CFI_ERR_NULL;
    *variant = choose_variant(layer, batch);
    return CFI_OK;
}

extern "C" cfi_status_t cfi_dense_tile_shape(const cfi_layer_t* layer, int32_t batch, int32_t* tile_n, int32_t* cluster) {
    if (!layer || !tile_n || !cluster) return CFI_ERR_NULL;
    if (!layer->tc_ok || batch < 1) return CFI_ERR_SHAPE;
    DeviceGuard g(layer->device);
    if (layer->dtype == CFI_BF16) {
        const bool persistent = tc_bf16_persistent(layer, batch);
        *tile_n = persistent ? kTpN : kTcN, *cluster = persistent ? 1 : tc_bf16_split(layer, batch);
    } else {
        const SplitShape sh = split_shape(layer, batch);
        if (!sh.ok) return CFI_ERR_SHAPE;
        *tile_n = sh.bt, *cluster = sh.split;
    }
    return CFI_OK;
}

extern "C" cfi_status_t cfi_forward_variant(const cfi_layer_t* layer, const void* x, void* y, int32_t batch,
                                            cfi_stream_t stream, cfi_variant_t variant) {
    if (!layer) return CFI_ERR_NULL;
    if (batch < 0) return CFI_ERR_SHAPE;
    if (batch == 0 || layer->d.out == 0) return CFI_OK;
    if (!y || (!x && layer->d.in > 0)) return CFI_ERR_NULL;
    if (((uintptr_t)x | (uintptr_t)y) & 15u) return CFI_ERR_ALIGNMENT;
    DeviceGuard g(layer->device);  // kernels, tensor maps and shared-memory opt-ins belong to the layer's device
    int v = variant;
    if (v == CFI_VARIANT_AUTO) v = choose_variant(layer, batch);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const bool bf = layer->dtype == CFI_BF16;
    switch (v) {
        case CFI_VARIANT_SIMPLE:
            return bf ? launch_simple<__nv_bfloat16>(layer, x, y, batch, st) : launch_simple<float>(layer, x, y, batch, st);
        case CFI_VARIANT_SPLITK: {
            const SplitkShape s = splitk_shape(layer, batch);
            return bf ? launch_splitk<__nv_bfloat16>(layer, s, x, y, batch, st)
                      : launch_splitk<float>(layer, s, x, y, batch, st);
        }
        case CFI_VARIANT_DENSE_TC:
            return launch_dense_tc(layer, x, y, batch, st);
        case CFI_VARIANT_SLAB:
            return bf ? launch_slab<__nv_bfloat16>(layer, x, y, batch, st) : launch_slab<float>(layer, x, y, batch, st);
        case CFI_VARIANT_BATCH: {
            const BatchShape s = batch_shape(layer, batch);
            return bf ? launch_batch<__nv_bfloat16>(layer, s, x, y, batch, st)
                      : launch_batch<float>(layer, s, x, y, batch, st);
        }
    }
    return CFI_ERR_DTYPE;
}

extern "C" cfi_status_t cfi_forward_dense(const cfi_layer_t* layer, const void* x, void* y, int32_t batch, cfi_stream_t stream,
                                          int32_t tile, int32_t cluster) {
    if (!layer) return CFI_ERR_NULL;
    if (batch < 0) return CFI_ERR_SHAPE;
    if (batch == 0 || layer->d.out == 0) return CFI_OK;
    if (!y || (!x && layer->d.in > 0)) return CFI_ERR_NULL;
    if (((uintptr_t)x | (uintptr_t)y) & 15u) return CFI_ERR_ALIGNMENT;
    DeviceGuard g(layer->device);
    return launch_dense_tc(layer, x, y, batch, reinterpret_cast<cudaStream_t>(stream), tile, cluster);
}

extern "C" cfi_status_t cfi_forward(const cfi_layer_t* layer, const void* x, void* y, int32_t batch,
                                    cfi_stream_t stream) {
    return cfi_forward_variant(layer, x, y, batch, stream, CFI_VARIANT_AUTO);
}

extern "C" cfi_status_t cfi_forward_host(cfi_layer_t* layer, const void* x_host, void* y_host, int32_t batch,
                                         cfi_stream_t stream) {
    if (!layer) return CFI_ERR_NULL;
    if (batch < 0) return CFI_ERR_SHAPE;
    if (batch == 0) return CFI_OK;
    if (!y_host || (!x_host && layer->d.in > 0)) return CFI_ERR_NULL;
    DeviceGuard g(layer->device);
    const size_t es = layer->dtype == CFI_BF16 ? 2 : 4;
    if (batch > layer->staged_batch) {
        if (layer->stage_x) cudaFree(layer->stage_x);
        if (layer->stage_y) cudaFree(layer->stage_y);
        layer->stage_x = layer->stage_y = nullptr;
        layer->staged_batch = 0;
        const size_t xb = std::max<size_t>((size_t)batch * layer->d.in * es, 16);
        const size_t yb = std::max<size_t>((size_t)batch * layer->d.out * es, 16);
        if (cudaMalloc(&layer->stage_x, xb) != cudaSuccess || cudaMalloc(&layer->stage_y, yb) != cudaSuccess) {
            cudaGetLastError();
            return CFI_ERR_ALLOC;
        }
        layer->staged_batch = batch;
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const size_t xb = (size_t)batch * layer->d.in * es, yb = (size_t)batch * layer->d.out * es;
    if (xb && cudaMemcpyAsync(layer->stage_x, x_host, xb, cudaMemcpyHostToDevice, st) != cudaSuccess) return CFI_ERR_CUDA;
    if (cfi_status_t e = cfi_forward(layer, layer->stage_x, layer->stage_y, batch, stream)) return e;
    if (yb && cudaMemcpyAsync(y_host, layer->stage_y, yb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return CFI_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? CFI_OK : CFI_ERR_CUDA;
}

extern "C" cfi_status_t cfi_layer_info(const cfi_layer_t* layer, cfi_layer_info_t* info) {
    if (!layer || !info) return CFI_ERR_NULL;
    const DevLayer& d = layer->d;
    const int64_t vs = layer->dtype == CFI_BF16 ? 2 : 4;
    info->in_features = d.in, info->out_features = d.out, info->n_active = d.n_active, info->k = d.k;
    info->dtype = layer->dtype, info->act = d.act;
    info->k_padded = d.kp;
    info->batch_slab_columns = d.cs;
    info->batch_row_stride = d.stride_q * 4;
    info->reserved = 0;
    info->weight_bytes_splitk = (int64_t)d.n_active * d.kp * (vs + (d.idx16 ? 2 : 4));
    info->weight_bytes_batch = (int64_t)d.n_active * d.stride_q * 32;
    info->device_bytes = layer->device_bytes;
    info->bytes_small_batch = layer->bytes_small;
    info->bytes_gather = layer->bytes_gather;
    info->bytes_dense = layer->bytes_dense;
    info->layouts = layer->layouts;
    info->reserved2 = 0;
    return CFI_OK;
}

extern "C" cfi_status_t cfi_device_status(const cfi_layer_t* layer, cfi_stream_t stream, int32_t* flag) {
    if (!layer || !flag) return CFI_ERR_NULL;
    DeviceGuard g(layer->device);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return CFI_ERR_CUDA;
    if (cudaMemcpy(flag, layer->d.status, sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess) return CFI_ERR_CUDA;
    return *flag ? CFI_ERR_DEVICE_FLAG : CFI_OK;
}

extern "C" cfi_status_t cfi_stack_create(cfi_layer_t* const* layers, int32_t n_layers, int32_t max_batch,
                                         cfi_stack_t** stack) {
    if (!stack) return CFI_ERR_NULL;
    *stack = nullptr;
    if (!layers) return CFI_ERR_NULL;
    if (n_layers < 1 || max_batch < 0) return CFI_ERR_SHAPE;
    for (int i = 0; i < n_layers; ++i) {
        if (!layers[i]) return CFI_ERR_NULL;
        if (layers[i]->dtype != layers[0]->dtype || layers[i]->device != layers[0]->device) return CFI_ERR_DTYPE;
        if (i && layers[i]->d.in != layers[i - 1]->d.out) return CFI_ERR_SHAPE;
    }
    cfi_stack* s = new (std::nothrow) cfi_stack();
    if (!s) return CFI_ERR_ALLOC;
    s->layers.assign(layers, layers + n_layers);
    s->max_batch = max_batch;
    s->dtype = layers[0]->dtype;
    int widest = 0;
    for (int i = 0; i + 1 < n_layers; ++i) widest = std::max(widest, layers[i]->d.out);
    const size_t es = s->dtype == CFI_BF16 ? 2 : 4;
    const size_t bytes = std::max<size_t>((size_t)max_batch * widest * es, 16);
    DeviceGuard g(layers[0]->device);
    for (int i = 0; i < 2; ++i)
        if (cudaMalloc(&s->buf[i], bytes) != cudaSuccess) {
            cudaGetLastError();
            cfi_stack_destroy(s);
            return CFI_ERR_ALLOC;
        }
    *stack = s;
    return CFI_OK;
}

extern "C" cfi_status_t cfi_stack_forward(const cfi_stack_t* stack, const void* x, void* y, int32_t batch,
                                          cfi_stream_t stream) {
    if (!stack) return CFI_ERR_NULL;
    if (batch < 0) return CFI_ERR_SHAPE;
    if (batch > stack->max_batch) return CFI_ERR_BUFFER_TOO_SMALL;
    const void* cur = x;
    const int n = (int)stack->layers.size();
    for (int i = 0; i < n; ++i) {
        void* dst = i + 1 == n ? y : stack->buf[i & 1];
        if (cfi_status_t e = cfi_forward(stack->layers[i], cur, dst, batch, stream)) return e;
        cur = dst;
    }
    return CFI_OK;
}

extern "C" cfi_status_t cfi_stack_destroy(cfi_stack_t* stack) {
    if (!stack) return CFI_OK;
    for (int i = 0; i < 2; ++i)
        if (stack->buf[i]) cudaFree(stack->buf[i]);
    delete stack;
    return CFI_OK;
}

// ------------------------------------------------------------------------------------------------
// Chain of layers without any allocation: the intermediates live in a fixed device array.
// ------------------------------------------------------------------------------------------------
namespace {

constexpr size_t kStaticScratchBytes = (size_t)8 << 20;  // two halves of 4 MiB, used alternately
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of g_static_scratch per device.  In host code the array's name only stands for the symbol;
// the address a kernel can use has to be asked for, with the owning device current.
std::atomic<unsigned char*> g_static_scratch_addr[kMaxDevices];

cfi_status_t static_scratch(int device, unsigned char** base) {
    if (device < 0 || device >= kMaxDevices) return CFI_ERR_SHAPE;
    unsigned char* p = g_static_scratch_addr[device].load(std::memory_order_acquire);
    if (!p) {
        void* sym = nullptr;
        if (cudaGetSymbolAddress(&sym, g_static_scratch) != cudaSuccess || !sym) {
            cudaGetLastError();
            return CFI_ERR_CUDA;
        }
        p = static_cast<unsigned char*>(sym);
        g_static_scratch_addr[device].store(p, std::memory_order_release);
    }
    *base = p;
    return CFI_OK;
}

}  // namespace

extern "C" cfi_status_t cfi_stack_forward_static(cfi_layer_t* const* layers, int32_t n_layers, const void* x, void* y,
                                                 int32_t batch, cfi_stream_t stream) {
    if (!layers) return CFI_ERR_NULL;
    if (n_layers < 1 || batch < 0) return CFI_ERR_SHAPE;
    size_t widest = 0;
    for (int i = 0; i < n_layers; ++i) {
        if (!layers[i]) return CFI_ERR_NULL;
        if (layers[i]->dtype != layers[0]->dtype || layers[i]->device != layers[0]->device) return CFI_ERR_DTYPE;
        if (i && layers[i]->d.in != layers[i - 1]->d.out) return CFI_ERR_SHAPE;
        if (i + 1 < n_layers) widest = std::max(widest, (size_t)layers[i]->d.out);
    }
    const size_t es = layers[0]->dtype == CFI_BF16 ? 2 : 4;
    if ((size_t)batch * widest * es > kStaticScratchBytes / 2) return CFI_ERR_BUFFER_TOO_SMALL;
    DeviceGuard g(layers[0]->device);
    unsigned char* base = nullptr;
    if (cfi_status_t e = static_scratch(layers[0]->device, &base)) return e;
    const void* cur = x;
    for (int i = 0; i < n_layers; ++i) {
        void* dst = i + 1 == n_layers ? y : base + (size_t)(i & 1) * (kStaticScratchBytes / 2);
        if (cfi_status_t e = cfi_forward(layers[i], cur, dst, batch, stream)) return e;
        cur = dst;
    }
    return CFI_OK;
}
