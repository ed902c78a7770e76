// cfi_srigl_update: one SRigL mask update of one layer on the device (Sec. 3.1, steps 1-7 "for each layer").
//
// Dense layout, as a training loop holds it: w[out][in] (zero where masked), mask[out][in] (0/1), grad[out][in].
// The update needs two selections over the whole layer -- the K smallest magnitudes among the active weights and the
// K largest gradient magnitudes among the inactive positions of live neurons -- and one selection per neuron (regrow
// to the new fan-in k', or trim down to it).  All of them are "the m smallest of a set of (32-bit key, position)
// pairs, ties to the smaller position", with key = the bits of |w| (a non-negative float orders like its bits) or
// the complement of the bits of |grad| (so that a larger gradient is a smaller key).  They are done by radix
// selection: four passes of 256-bin histograms over the digits of the key from the top, each pass narrowing to the
// bin that holds the m-th element, then the ties on the final key are cut in position order.  For the two layer-wide
// selections the last pass also lists the few elements that match the first three digits; when a list holds them all
// (the rule), the position of the last tie taken is selected from it and the marking pass is elementwise; inputs with
// very many equal keys overflow the list and are ranked with per-chunk tie counts and a prefix sum instead.
//
// Readings where Sec. 3.1 leaves a choice (the same as the CPU oracle used by the tests takes): already ablated
// neurons stay out; a weight is salient if it is active and not among the K smallest, or inactive and among the K
// largest gradients; a neuron is ablated if its salient count is below max(1, gamma_sal * k);
// k' = min(in, floor(k * live_before / live_after)); step 7 may regrow any position of the neuron that is not active
// at that moment (a weight pruned in step 6 included; grown weights start at 0); a neuron left with more than k'
// weights after step 6 loses its smallest down to k'.
#include "cfi.h"

#include <cuda_runtime.h>

#include <cstdint>

namespace {

constexpr int kThreads = 256, kChunk = 16 * kThreads;  // a block marks ties over 4096 consecutive positions

struct SelectState {
    unsigned long long want;     // elements still to take inside the current prefix bin (1-based rank of the cut)
    unsigned long long below;    // elements with a key below the current prefix
    unsigned int prefix, prefix_mask;
    unsigned int hist[256];
    unsigned int blocks_done;    // blocks of the running histogram sweep that have added their counts (first state only)
    // The last sweep also lists the elements that match the first three digits (key, position): a few hundred as a rule.
    // If the list holds them all, the position of the last tie taken follows from it and the marking needs no ranking.
    unsigned int listed;         // elements offered to the list (may exceed its capacity)
    unsigned int last_tie;       // ties on the cut key are taken up to and including this position
    unsigned int listed_all;     // 1: last_tie is valid
};

// Capacity of a selection's list: enough for ordinary key distributions, small against the layer; inputs with very many
// equal keys overflow it and take the ranking path.
__host__ __device__ inline unsigned int list_capacity(long long n) {
    const long long c = n / 64;
    return (unsigned int)(c < 64 ? 64 : c > 32768 ? 32768 : c);
}

struct Scalars {
    long long active_total, inactive_total;
    int k, k_new, live_before, live_after;
};

__device__ __forceinline__ unsigned int mag_bits(float v) { return __float_as_uint(fabsf(v)); }

// h[bin] += 1 for every lane that takes part; lanes of the warp with the same bin are counted by one of them.  (The top
// digits of float magnitudes fall into a handful of bins, and a plain atomic per lane would serialise on them.)
__device__ __forceinline__ void hist_add(unsigned int* h, bool take, unsigned int bin) {
    const unsigned int active = __ballot_sync(0xffffffffu, take);
    if (take) {
        const unsigned int peers = __match_any_sync(active, bin);
        if ((int)(__ffs(peers) - 1) == (int)(threadIdx.x & 31)) atomicAdd(&h[bin], (unsigned int)__popc(peers));
    }
}

__global__ void row_count_kernel(const uint8_t* mask, int out_f, int in_f, int* row_count) {
    __shared__ int s;
    const int r = blockIdx.x;
    if (threadIdx.x == 0) s = 0;
    __syncthreads();
    int c = 0;
    if ((in_f & 15) == 0) {  // 16 mask bytes per load; __vcmpne4 turns every nonzero byte into 0xff
        const uint4* m16 = reinterpret_cast<const uint4*>(mask + (size_t)r * in_f);
        for (int v = threadIdx.x; v < (in_f >> 4); v += blockDim.x) {
            const uint4 m = m16[v];
            c += (__popc(__vcmpne4(m.x, 0u)) + __popc(__vcmpne4(m.y, 0u)) + __popc(__vcmpne4(m.z, 0u)) + __popc(__vcmpne4(m.w, 0u))) >> 3;
        }
    } else {
        for (int j = threadIdx.x; j < in_f; j += blockDim.x) c += mask[(size_t)r * in_f + j] ? 1 : 0;
    }
    for (int off = 16; off > 0; off >>= 1) c += __shfl_down_sync(0xffffffffu, c, off);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(&s, c);
    __syncthreads();
    if (threadIdx.x == 0) row_count[r] = s;
}

// Single block: totals, k, and the initial state of the two layer-wide selections (K clipped to both pools).
__global__ void setup_kernel(const int* row_count, int out_f, int in_f, long long K, Scalars* sc, SelectState* st) {
    __shared__ long long act;
    __shared__ int live, k;
    if (threadIdx.x == 0) act = 0, live = 0, k = 0;
    __syncthreads();
    long long my_act = 0;
    int my_live = 0, my_k = 0;
    for (int r0 = threadIdx.x; r0 < out_f; r0 += 8 * blockDim.x) {  // eight rows' loads in flight
        int rc[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) rc[u] = r0 + u * blockDim.x < out_f ? row_count[r0 + u * blockDim.x] : 0;
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (rc[u] > 0) my_act += rc[u], ++my_live, my_k = max(my_k, rc[u]);
    }
    for (int off = 16; off > 0; off >>= 1) {  // one set of atomics per warp
        my_act += __shfl_down_sync(0xffffffffu, my_act, off);
        my_live += __shfl_down_sync(0xffffffffu, my_live, off);
        my_k = max(my_k, __shfl_down_sync(0xffffffffu, my_k, off));
    }
    if ((threadIdx.x & 31) == 0 && my_live) {
        atomicAdd((unsigned long long*)&act, (unsigned long long)my_act);
        atomicAdd(&live, my_live);
        atomicMax(&k, my_k);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        sc->active_total = act;
        sc->inactive_total = (long long)live * in_f - act;
        sc->k = k, sc->live_before = live, sc->k_new = 0, sc->live_after = 0;
        long long kk = K < 0 ? 0 : K;
        if (kk > act) kk = act;
        if (kk > sc->inactive_total) kk = sc->inactive_total;
        for (int s = 0; s < 2; ++s)
            st[s].want = (unsigned long long)kk, st[s].below = 0, st[s].prefix = 0, st[s].prefix_mask = 0, st[s].blocks_done = 0,
            st[s].listed = 0, st[s].last_tie = 0, st[s].listed_all = 0;
    }
    for (int s = 0; s < 2; ++s)
        for (int b = threadIdx.x; b < 256; b += blockDim.x) st[s].hist[b] = 0;
}

// One warp per selection: the bin that holds the `want`-th element (the first bin whose running count reaches it;
// the last bin if none before it does); narrow the prefix to it and clear the histogram for the next pass.  Called by
// the last block of a histogram sweep, after every block's counts have arrived.
__device__ void pick_bin(int pass, SelectState* st) {
    const int lane = threadIdx.x & 31;
    const unsigned long long want = st->want;
    unsigned int v[8];
    unsigned long long mine = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = __ldcg(&st->hist[8 * lane + e]), mine += v[e];
    unsigned long long incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += up;
    }
    unsigned long long seen = incl - mine;  // count in the bins before this lane's
    int found = 256;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        if (found == 256) {
            if (seen + v[e] >= want) found = 8 * lane + e;
            else seen += v[e];
        }
    }
    int bin = found;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) bin = min(bin, __shfl_xor_sync(0xffffffffu, bin, off));
    if (bin > 255) bin = 255;
    // `seen` of the lane that owns the bin is the count below it (for the last bin without a hit: lane 31 stopped there)
    if (found == 256 && lane == 31) seen -= v[7];
    const unsigned long long below_bin = __shfl_sync(0xffffffffu, seen, bin >> 3);
#pragma unroll
    for (int e = 0; e < 8; ++e) st->hist[8 * lane + e] = 0;
    if (lane == 0 && want != 0) {
        const int shift = 24 - 8 * pass;
        st->want = want - below_bin;
        st->below += below_bin;
        st->prefix |= (unsigned int)bin << shift;
        st->prefix_mask |= 255u << shift;
    }
}

// The whole block (kThreads threads), one selection, after its last digit has been picked: if the list holds every
// element that matched the first three digits, the ties on the cut key are all in it, and the position of the last tie
// taken (the `want`-th in position order) is found by radix selection over the listed positions.  Then "taken" is
// key < cut, or key == cut and position <= last_tie: the marking needs neither tie counts nor ranks.
__device__ void find_last_tie(SelectState* st, const uint2* list, unsigned int cap) {
    __shared__ unsigned int hist[256], warp_tot[kThreads / 32], res[2], ties_total;
    const int t = threadIdx.x, lane = t & 31, wid = t >> 5;
    const unsigned int n = __ldcg(&st->listed);
    if (n > cap) {  // the list overflowed (the same for the whole block): the ranking path decides
        if (t == 0) st->listed_all = 0;
        return;
    }
    const unsigned int cut = __ldcg(&st->prefix);
    unsigned int want = (unsigned int)__ldcg(&st->want);  // ties to take
    if (t == 0) ties_total = 0;
    __syncthreads();
    unsigned int mine = 0;
    for (unsigned int i = t; i < n; i += kThreads) mine += __ldcg(&list[i]).x == cut ? 1u : 0u;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mine += __shfl_down_sync(0xffffffffu, mine, off);
    if (lane == 0 && mine) atomicAdd(&ties_total, mine);
    __syncthreads();
    if (want == 0 || ties_total <= want) {  // selection off, or every tie is taken
        if (t == 0) st->last_tie = 0xFFFFFFFFu, st->listed_all = 1;
        return;
    }
    unsigned int prefix = 0, pmask = 0;
    for (int pass = 0; pass < 4; ++pass) {
        hist[t] = 0;
        __syncthreads();
        const int shift = 24 - 8 * pass;
        for (unsigned int i = t; i < n; i += kThreads) {
            const uint2 e = __ldcg(&list[i]);
            if (e.x == cut && (e.y & pmask) == prefix) atomicAdd(&hist[(e.y >> shift) & 255u], 1u);
        }
        __syncthreads();
        const unsigned int h = hist[t];
        unsigned int incl = h;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned int up = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += up;
        }
        if (lane == 31) warp_tot[wid] = incl;
        __syncthreads();
        unsigned int before = 0;
#pragma unroll
        for (int i = 0; i < kThreads / 32; ++i) before += i < wid ? warp_tot[i] : 0u;
        const unsigned int excl = before + incl - h;
        if (excl < want && want <= excl + h) res[0] = (unsigned int)t, res[1] = excl;  // exactly one thread: want <= ties
        __syncthreads();
        prefix |= res[0] << shift;
        pmask |= 255u << shift;
        want -= res[1];
        __syncthreads();  // res[] and hist[] are rewritten by the next pass
    }
    if (t == 0) st->last_tie = prefix, st->listed_all = 1;
}

// Histograms of digit `pass` (0 = top byte) for both layer-wide selections in one sweep over the layer: over the valid
// elements of each whose key matches the prefix found so far.  Every position is valid for at most one of the two, so
// one histogram of 512 bins (selection * 256 + digit) serves both.  A block takes whole rows, four columns per thread
// and step when the row length is a multiple of four (16-byte loads of w and grad, 4-byte loads of the mask).
template <bool LAST>  // the last sweep (pass 3) also fills the lists; the others keep their smaller code
__global__ void __launch_bounds__(kThreads, 8) hist_kernel(const float* w, const uint8_t* mask, const float* grad, const int* row_count, int out_f, int in_f,
                            int pass, SelectState* st, uint2* list, unsigned int cap) {
    __shared__ unsigned int h[512];
    __shared__ int list_full[2];
    if (threadIdx.x < 2) list_full[threadIdx.x] = 0;
    for (int b = threadIdx.x; b < 512; b += blockDim.x) h[b] = 0;
    __syncthreads();
    const bool on0 = st[0].want != 0, on1 = st[1].want != 0;
    if (on0 || on1) {
        const unsigned int prefix0 = st[0].prefix, pmask0 = st[0].prefix_mask, prefix1 = st[1].prefix, pmask1 = st[1].prefix_mask;
        const int shift = 24 - 8 * pass;
        auto one = [&](bool inside, uint8_t m, float wv, float gv, size_t pos) {  // every lane of the warp calls it the same number of times
            bool take = false;
            unsigned int bin = 0;
            if (inside) {
                const unsigned int key = m ? mag_bits(wv) : ~mag_bits(gv);
                take = m ? (on0 && (key & pmask0) == prefix0) : (on1 && (key & pmask1) == prefix1);
                bin = (m ? 0u : 256u) + ((key >> shift) & 255u);
                if (LAST && take) {  // the last sweep lists what it counts, while the list has room
                    const int sel = m ? 0 : 1;
                    if (!list_full[sel]) {
                        const unsigned int at = atomicAdd(&st[sel].listed, 1u);
                        if (at < cap) list[(size_t)sel * cap + at] = make_uint2(key, (unsigned int)pos);
                        else list_full[sel] = 1;
                    }
                }
            }
            // The top digit falls into a handful of bins (aggregate per warp); the later digits of the few elements that
            // still match the prefix spread out, and a plain atomic is cheaper there.
            if (pass == 0) hist_add(h, take, bin);
            else if (take) atomicAdd(&h[bin], 1u);
        };
        for (int r = blockIdx.x; r < out_f; r += gridDim.x) {
            if (row_count[r] == 0) continue;  // a neuron without weights is in neither pool
            const size_t base = (size_t)r * in_f;
            if ((in_f & 3) == 0) {
                const uchar4* m4 = reinterpret_cast<const uchar4*>(mask + base);
                const float4* w4 = reinterpret_cast<const float4*>(w + base);
                const float4* g4 = reinterpret_cast<const float4*>(grad + base);
                const int n4 = in_f >> 2;
                for (int v0 = 0; v0 < n4; v0 += blockDim.x) {
                    const int v = v0 + threadIdx.x;
                    const bool inside = v < n4;
                    uchar4 m = make_uchar4(0, 0, 0, 0);
                    float4 wv = make_float4(0.f, 0.f, 0.f, 0.f), gv = wv;
                    if (inside) {  // all three at once: a load that waited for the mask would cost a second trip to memory
                        m = m4[v];
                        wv = w4[v];
                        gv = g4[v];
                    }
                    one(inside, m.x, wv.x, gv.x, base + 4 * (size_t)v);
                    one(inside, m.y, wv.y, gv.y, base + 4 * (size_t)v + 1);
                    one(inside, m.z, wv.z, gv.z, base + 4 * (size_t)v + 2);
                    one(inside, m.w, wv.w, gv.w, base + 4 * (size_t)v + 3);
                }
            } else {
                for (int c0 = 0; c0 < in_f; c0 += blockDim.x) {
                    const int c = c0 + threadIdx.x;
                    const bool inside = c < in_f;
                    const uint8_t m = inside ? mask[base + c] : 0;
                    one(inside, m, inside && m ? w[base + c] : 0.f, inside && !m ? grad[base + c] : 0.f, base + c);
                }
            }
        }
    }
    __syncthreads();
    for (int b = threadIdx.x; b < 512; b += blockDim.x)
        if (h[b]) atomicAdd(&st[b >> 8].hist[b & 255], h[b]);
    // The block whose counts arrive last narrows both selections to their bins (no separate launch, nobody waits).
    __shared__ bool last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(&st[0].blocks_done, 1u) == gridDim.x - 1;
    __syncthreads();
    if (last) {
        __threadfence();
        if (threadIdx.x < 64) pick_bin(pass, st + (threadIdx.x >> 5));
        if (LAST) {  // both cuts are final
            __syncthreads();
            find_last_tie(st, list, cap);
            __syncthreads();
            find_last_tie(st + 1, list + cap, cap);
        }
        if (threadIdx.x == 0) st[0].blocks_done = 0;
    }
}

// A thread's run of 16 consecutive positions from `base`: kind (0: in neither pool, 1: active weight, 2: inactive position
// of a live neuron) and key of each.  When the run lies inside one row and the arrays allow 16-byte loads it takes one
// load of the 16 mask bytes and four 16-byte loads each of the weights and the gradients, all requested together.
__device__ __forceinline__ void load_run16(const float* w, const uint8_t* mask, const float* grad, const int* row_count, int in_f,
                                           long long n, long long base, bool vec_ok, unsigned int (&keys)[16], uint8_t (&kind)[16]) {
    if (vec_ok && base + 16 <= n) {
        // Everything is requested at once: a load that waited for the mask would cost a second trip to memory.
        const uint4 m16 = *reinterpret_cast<const uint4*>(mask + base);
        float4 w16[4], g16[4];
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            w16[g] = *reinterpret_cast<const float4*>(w + base + 4 * g);
            g16[g] = *reinterpret_cast<const float4*>(grad + base + 4 * g);
        }
        const unsigned int mw[4] = {m16.x, m16.y, m16.z, m16.w};
        const bool live = row_count[(unsigned int)((unsigned long long)base / (unsigned int)in_f)] != 0;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const unsigned int nz = __vcmpne4(mw[g], 0u);  // 0xff per nonzero mask byte
            const float4 wv = w16[g], gv = g16[g];
            const float we[4] = {wv.x, wv.y, wv.z, wv.w}, ge[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool on = ((nz >> (8 * e)) & 1u) != 0u;
                kind[4 * g + e] = on ? 1 : live ? 2 : 0;
                keys[4 * g + e] = on ? mag_bits(we[e]) : live ? ~mag_bits(ge[e]) : 0u;
            }
        }
        return;
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        kind[e] = 0, keys[e] = 0;
        const long long p = base + e;
        if (p < n) {
            if (mask[p]) kind[e] = 1, keys[e] = mag_bits(w[p]);
            else if (row_count[(unsigned int)((unsigned long long)p / (unsigned int)in_f)] != 0) kind[e] = 2, keys[e] = ~mag_bits(grad[p]);
        }
    }
}

// After the four passes prefix is the key of the cut and `want` of the elements equal to it are taken, the first ones
// in position order.  Per chunk of kChunk positions and per selection: how many equal the cut key.
__global__ void tie_count_kernel(const float* w, const uint8_t* mask, const float* grad, const int* row_count, int in_f,
                                 long long n, const SelectState* st, unsigned int* chunk_ties, int n_chunks, bool vec_ok) {
    __shared__ unsigned int s[2];
    if (st[0].listed_all && st[1].listed_all) return;  // the marking will not ask for tie counts
    if (threadIdx.x < 2) s[threadIdx.x] = 0;
    __syncthreads();
    const long long base = (long long)blockIdx.x * kChunk + (long long)threadIdx.x * 16;
    const bool on0 = st[0].want != 0, on1 = st[1].want != 0;
    const unsigned int cut0 = st[0].prefix, cut1 = st[1].prefix;
    unsigned int c0 = 0, c1 = 0;
    unsigned int keys[16];
    uint8_t kind[16];
    load_run16(w, mask, grad, row_count, in_f, n, base, vec_ok, keys, kind);
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        c0 += (kind[e] == 1 && on0 && keys[e] == cut0) ? 1u : 0u;
        c1 += (kind[e] == 2 && on1 && keys[e] == cut1) ? 1u : 0u;
    }
    if (c0) atomicAdd(&s[0], c0);
    if (c1) atomicAdd(&s[1], c1);
    __syncthreads();
    if (threadIdx.x < 2) chunk_ties[(size_t)threadIdx.x * n_chunks + blockIdx.x] = s[threadIdx.x];
}

// One block per selection: exclusive prefix sum of its per-chunk tie counts, in place.
__global__ void chunk_scan_kernel(unsigned int* chunk_ties_both, int n_chunks, const SelectState* st) {
    if (st[0].listed_all && st[1].listed_all) return;
    unsigned int* chunk_ties = chunk_ties_both + (size_t)blockIdx.x * n_chunks;
    __shared__ unsigned long long warp_tot[kThreads / 32];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    // A thread takes 16 consecutive chunks at a time (the block 4096): their sum is scanned over the block with shuffles
    // and one count per warp, then the thread walks its chunks.
    unsigned long long carry = 0;
    for (int c0 = 0; c0 < n_chunks; c0 += 16 * kThreads) {
        const int first = c0 + 16 * threadIdx.x;
        unsigned int v[16];
        unsigned long long mine = 0;
#pragma unroll
        for (int e = 0; e < 16; ++e) v[e] = first + e < n_chunks ? chunk_ties[first + e] : 0u, mine += v[e];
        unsigned long long incl = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += up;
        }
        if (lane == 31) warp_tot[wid] = incl;
        __syncthreads();
        unsigned long long before = carry + incl - mine, total = 0;
#pragma unroll
        for (int i = 0; i < kThreads / 32; ++i) {
            const unsigned long long p = warp_tot[i];
            before += i < wid ? p : 0ull;
            total += p;
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            if (first + e < n_chunks) chunk_ties[first + e] = (unsigned int)(before > 0xFFFFFFFFull ? 0xFFFFFFFFull : before);
            before += v[e];
        }
        carry += total;
        __syncthreads();  // warp_tot[] is rewritten by the next round
    }
}

// drop[p] / grow_top[p] = 1 for the selected elements of the two selections: key below the cut, or equal to it and among
// the first `want` in position order.
__global__ void mark_kernel(const float* w, const uint8_t* mask, const float* grad, const int* row_count, int in_f, long long n,
                            const SelectState* st, const unsigned int* chunk_ties, int n_chunks, uint8_t* drop,
                            uint8_t* grow_top, bool vec_ok) {
    __shared__ unsigned int part[2][kThreads];
    const long long base = (long long)blockIdx.x * kChunk + (long long)threadIdx.x * 16;
    const unsigned long long want0 = st[0].want, want1 = st[1].want;
    const unsigned int cut0 = st[0].prefix, cut1 = st[1].prefix;
    unsigned int keys[16];
    uint8_t kind[16];  // 0: in neither pool, 1: active weight, 2: inactive position of a live neuron
    unsigned int mine0 = 0, mine1 = 0;
    load_run16(w, mask, grad, row_count, in_f, n, base, vec_ok, keys, kind);
    unsigned int d16[4] = {0u, 0u, 0u, 0u}, g16[4] = {0u, 0u, 0u, 0u};  // the 16 flags of each kind, one byte each
    if (st[0].listed_all && st[1].listed_all) {
        // Both lists held every candidate of the last digit: a tie is taken up to a known position, nothing to rank.
        const unsigned int last0 = st[0].last_tie, last1 = st[1].last_tie;
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const unsigned int pos = (unsigned int)(base + e);
            const unsigned int f0 = (kind[e] == 1 && want0 != 0 && (keys[e] < cut0 || (keys[e] == cut0 && pos <= last0))) ? 1u : 0u;
            const unsigned int f1 = (kind[e] == 2 && want1 != 0 && (keys[e] < cut1 || (keys[e] == cut1 && pos <= last1))) ? 1u : 0u;
            d16[e >> 2] |= f0 << (8 * (e & 3));
            g16[e >> 2] |= f1 << (8 * (e & 3));
        }
    } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            if (kind[e] == 1 && want0 != 0 && keys[e] == cut0) ++mine0;
            if (kind[e] == 2 && want1 != 0 && keys[e] == cut1) ++mine1;
        }
        part[0][threadIdx.x] = mine0;
        part[1][threadIdx.x] = mine1;
        __syncthreads();
        for (int off = 1; off < kThreads; off <<= 1) {
            const unsigned int add0 = threadIdx.x >= off ? part[0][threadIdx.x - off] : 0u;
            const unsigned int add1 = threadIdx.x >= off ? part[1][threadIdx.x - off] : 0u;
            __syncthreads();
            part[0][threadIdx.x] += add0;
            part[1][threadIdx.x] += add1;
            __syncthreads();
        }
        // ties of each selection before this thread's first element
        unsigned long long rank0 = (unsigned long long)chunk_ties[blockIdx.x] + part[0][threadIdx.x] - mine0;
        unsigned long long rank1 = (unsigned long long)chunk_ties[(size_t)n_chunks + blockIdx.x] + part[1][threadIdx.x] - mine1;
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            unsigned int f0 = 0, f1 = 0;
            if (kind[e] == 1 && want0 != 0) {
                if (keys[e] < cut0) f0 = 1;
                else if (keys[e] == cut0) f0 = rank0++ < want0 ? 1 : 0;
            } else if (kind[e] == 2 && want1 != 0) {
                if (keys[e] < cut1) f1 = 1;
                else if (keys[e] == cut1) f1 = rank1++ < want1 ? 1 : 0;
            }
            d16[e >> 2] |= f0 << (8 * (e & 3));
            g16[e >> 2] |= f1 << (8 * (e & 3));
        }
    }
    if (vec_ok && base + 16 <= n) {
        *reinterpret_cast<uint4*>(drop + base) = make_uint4(d16[0], d16[1], d16[2], d16[3]);
        *reinterpret_cast<uint4*>(grow_top + base) = make_uint4(g16[0], g16[1], g16[2], g16[3]);
    } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            if (base + e >= n) continue;
            drop[base + e] = (uint8_t)((d16[e >> 2] >> (8 * (e & 3))) & 1u);
            grow_top[base + e] = (uint8_t)((g16[e >> 2] >> (8 * (e & 3))) & 1u);
        }
    }
}

// Step 3: salient weights per neuron.
__global__ void salient_kernel(const uint8_t* mask, const uint8_t* drop, const uint8_t* grow_top, int in_f, int* salient) {
    __shared__ int s;
    const int r = blockIdx.x;
    if (threadIdx.x == 0) s = 0;
    __syncthreads();
    int c = 0;
    const size_t base = (size_t)r * in_f;
    if ((in_f & 15) == 0 && (reinterpret_cast<uintptr_t>(mask) & 15u) == 0) {  // (the flag arrays are 256-byte aligned)
        const uint4 *m16 = reinterpret_cast<const uint4*>(mask + base), *d16 = reinterpret_cast<const uint4*>(drop + base),
                    *g16 = reinterpret_cast<const uint4*>(grow_top + base);
        for (int v = threadIdx.x; v < (in_f >> 4); v += blockDim.x) {
            const uint4 m = m16[v], d = d16[v], g = g16[v];
            // a byte is salient if (mask set and not dropped) or among the top gradients
            c += (__popc((__vcmpne4(m.x, 0u) & __vcmpeq4(d.x, 0u)) | __vcmpne4(g.x, 0u)) +
                  __popc((__vcmpne4(m.y, 0u) & __vcmpeq4(d.y, 0u)) | __vcmpne4(g.y, 0u)) +
                  __popc((__vcmpne4(m.z, 0u) & __vcmpeq4(d.z, 0u)) | __vcmpne4(g.z, 0u)) +
                  __popc((__vcmpne4(m.w, 0u) & __vcmpeq4(d.w, 0u)) | __vcmpne4(g.w, 0u))) >> 3;
        }
    } else if ((in_f & 3) == 0) {
        const uchar4 *m4 = reinterpret_cast<const uchar4*>(mask + base), *d4 = reinterpret_cast<const uchar4*>(drop + base),
                     *g4 = reinterpret_cast<const uchar4*>(grow_top + base);
        for (int v = threadIdx.x; v < (in_f >> 2); v += blockDim.x) {
            const uchar4 m = m4[v], d = d4[v], g = g4[v];
            c += ((m.x && !d.x) || g.x) + ((m.y && !d.y) || g.y) + ((m.z && !d.z) || g.z) + ((m.w && !d.w) || g.w);
        }
    } else {
        for (int j = threadIdx.x; j < in_f; j += blockDim.x)
            c += ((mask[base + j] && !drop[base + j]) || grow_top[base + j]) ? 1 : 0;
    }
    atomicAdd(&s, c);
    __syncthreads();
    if (threadIdx.x == 0) salient[r] = s;
}

// Steps 4 and 5 (single block): who is ablated, and the new fan-in.
__global__ void ablate_kernel(const int* row_count, const int* salient, int out_f, int in_f, float gamma_sal, Scalars* sc,
                              uint8_t* survives) {
    __shared__ int after;
    if (threadIdx.x == 0) after = 0;
    __syncthreads();
    const double threshold = fmax(1.0, (double)gamma_sal * (double)sc->k);
    int mine = 0;
    for (int r0 = threadIdx.x; r0 < out_f; r0 += 8 * blockDim.x) {  // eight rows' loads in flight: one block walks all rows
        int rc[8], sa[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int r = r0 + u * blockDim.x;
            rc[u] = r < out_f ? row_count[r] : 0, sa[u] = r < out_f ? salient[r] : 0;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int r = r0 + u * blockDim.x;
            if (r < out_f) {
                const bool live = rc[u] > 0 && !((double)sa[u] < threshold);
                survives[r] = live ? 1 : 0;
                mine += live ? 1 : 0;
            }
        }
    }
    for (int off = 16; off > 0; off >>= 1) mine += __shfl_down_sync(0xffffffffu, mine, off);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&after, mine);
    __syncthreads();
    if (threadIdx.x == 0) {
        sc->live_after = after;
        long long kn = after > 0 ? ((long long)sc->k * sc->live_before) / after : 0;
        if (kn > in_f) kn = in_f;
        sc->k_new = (int)kn;
    }
}

// Block-wide selection inside one row: the `m` smallest keys (ties to the smaller column) among the columns for which
// `key_of` returns true.  Returns through shared memory the cut key and how many ties on it to take; `take(c, key)`
// then answers for a column in increasing column order within the calling pattern below.
struct RowCut {
    unsigned int cut;
    unsigned int ties;   // elements equal to the cut to take, the first ones in column order
    int any;             // 0: nothing to select
};

// `count(prefix, prefix_mask, shift)` adds to hist[(key >> shift) & 255], with shared-memory atomics, every candidate of
// the row whose key matches the prefix found so far.
template <typename Count>
__device__ void row_select(int m, Count count, unsigned int* hist /*256, shared*/, RowCut* out /*shared*/) {
    __shared__ unsigned int prefix, pmask, want, warp_tot[kThreads / 32];
    if (threadIdx.x == 0) prefix = 0, pmask = 0, want = (unsigned int)(m > 0 ? m : 0);
    __syncthreads();
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int pass = 0; pass < 4 && m > 0; ++pass) {
        for (int b = threadIdx.x; b < 256; b += blockDim.x) hist[b] = 0;
        __syncthreads();
        const int shift = 24 - 8 * pass;
        count(prefix, pmask, shift);
        __syncthreads();
        // The bin that holds the `want`-th element, by the whole block (one bin per thread): the first bin whose running
        // count reaches `want`, the last bin if none does.  A prefix count over the block (shuffles, then one count per
        // warp); exactly one thread finds that the running count first reaches `want` in its bin.
        {
            const unsigned int h = hist[threadIdx.x], w0 = want;
            unsigned int incl = h;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned int up = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += up;
            }
            if (lane == 31) warp_tot[wid] = incl;
            __syncthreads();
            unsigned int before = 0, total = 0;
#pragma unroll
            for (int i = 0; i < kThreads / 32; ++i) {
                const unsigned int p = warp_tot[i];
                before += i < wid ? p : 0u;
                total += p;
            }
            const unsigned int excl = before + incl - h;
            const bool here = excl < w0 && w0 <= excl + h;
            const bool last_none = w0 > total && threadIdx.x == kThreads - 1;
            __syncthreads();  // every thread has read `want`
            if (here || last_none) {
                want = w0 - excl;
                prefix |= (unsigned int)threadIdx.x << shift;
                pmask |= 255u << shift;
            }
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) out->cut = prefix, out->ties = want, out->any = m > 0 ? 1 : 0;
    __syncthreads();
}

// Steps 6 and 7 for one neuron per block: prune, then trim or regrow to k'.  The row's keys for the selection that turns
// out to be needed (magnitudes of the kept weights when trimming, complemented gradient magnitudes of the free positions
// when regrowing) are put in shared memory once, next to a byte per column that says whether the column is kept, so
// that every 32-bit key value stays usable.  CACHED = false reads the operands from global memory on every pass
// instead (rows too long for shared memory).
template <bool CACHED>
__global__ void finalize_kernel(float* w, uint8_t* mask, const float* grad, const uint8_t* drop, const uint8_t* survives,
                                int in_f, const Scalars* sc) {
    extern __shared__ __align__(16) unsigned char row_smem[];  // CACHED: keys[in_f] (4 bytes each), then state[in_f] (1 byte each)
    __shared__ unsigned int hist[256];
    __shared__ RowCut cut;
    __shared__ int kept_count;
    __shared__ unsigned int part[kThreads / 32];
    const int r = blockIdx.x;
    float* wr = w + (size_t)r * in_f;
    uint8_t* mr = mask + (size_t)r * in_f;
    const float* gr = grad + (size_t)r * in_f;
    const uint8_t* dr = drop + (size_t)r * in_f;
    if (!survives[r]) {  // ablated now or before: nothing left
        for (int c = threadIdx.x; c < in_f; c += blockDim.x) wr[c] = 0.0f, mr[c] = 0;
        return;
    }
    unsigned int* keys = reinterpret_cast<unsigned int*>(row_smem);
    uint8_t* state = row_smem + (size_t)in_f * 4;  // 1 = kept after step 6, 0 = free
    const int k_new = sc->k_new;
    if (threadIdx.x == 0) kept_count = 0;
    __syncthreads();
    int mine = 0;
    for (int c = threadIdx.x; c < in_f; c += blockDim.x) {
        const bool is_kept = mr[c] && !dr[c];
        if (CACHED) state[c] = is_kept ? 1 : 0;
        mine += is_kept ? 1 : 0;
    }
    atomicAdd(&kept_count, mine);
    __syncthreads();
    const int kept = kept_count;
    const bool trim = kept > k_new;
    const int m = trim ? kept - k_new : k_new - kept;
    if (CACHED && m > 0) {
        for (int c = threadIdx.x; c < in_f; c += blockDim.x) {
            const bool candidate = trim ? state[c] != 0 : state[c] == 0;
            keys[c] = candidate ? (trim ? mag_bits(wr[c]) : ~mag_bits(gr[c])) : 0u;
        }
        __syncthreads();
    }
    auto key_of = [&](int c, unsigned int& key) {
        if (CACHED) {
            key = keys[c];
            return trim ? state[c] != 0 : state[c] == 0;
        }
        const bool is_kept = mr[c] && !dr[c];
        key = trim ? mag_bits(wr[c]) : ~mag_bits(gr[c]);
        return trim ? is_kept : !is_kept;
    };
    // trim: the kept weights with the smallest magnitudes go; otherwise the free positions with the largest gradient
    // magnitudes come
    row_select(m, [&](unsigned int pre, unsigned int pm, int shift) {
        for (int c = threadIdx.x; c < in_f; c += blockDim.x) {
            unsigned int key;
            if (key_of(c, key) && (key & pm) == pre) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        }
    }, hist, &cut);
    // Apply, walking the row in column order so that ties on the cut key go to the smaller columns: a tie's rank is
    // the ties of the chunks before (carried by every thread), of the warps before in this chunk (one count per warp
    // in shared memory) and of the lanes before in its warp (a ballot).
    unsigned int carry = 0;
    for (int c0 = 0; c0 < in_f; c0 += kThreads) {
        const int c = c0 + threadIdx.x;
        bool is_kept = false, candidate = false;
        unsigned int key = 0;
        if (c < in_f) {
            is_kept = CACHED ? state[c] != 0 : (mr[c] && !dr[c]);
            candidate = trim ? is_kept : !is_kept;
            if (cut.any && candidate) key = CACHED ? keys[c] : (trim ? mag_bits(wr[c]) : ~mag_bits(gr[c]));
        }
        const unsigned int tie = (cut.any && candidate && key == cut.cut) ? 1u : 0u;
        const unsigned int ties_in_warp = __ballot_sync(0xffffffffu, tie != 0);
        const int wid = threadIdx.x >> 5, ln = threadIdx.x & 31;
        if (ln == 0) part[wid] = (unsigned int)__popc(ties_in_warp);
        __syncthreads();
        unsigned int rank = carry + (unsigned int)__popc(ties_in_warp & ((1u << ln) - 1u)), in_chunk = 0;
#pragma unroll
        for (int i = 0; i < kThreads / 32; ++i) {
            const unsigned int p = part[i];
            rank += i < wid ? p : 0u;
            in_chunk += p;
        }
        if (c < in_f) {
            const bool selected = cut.any && candidate && (key < cut.cut || (tie && rank < cut.ties));
            bool on;
            if (trim) on = is_kept && !selected;
            else on = is_kept || selected;
            if (!on || !is_kept) wr[c] = 0.0f;  // pruned, trimmed, free, or grown (starts at 0); a survivor keeps its value
            mr[c] = on ? 1 : 0;
        }
        carry += in_chunk;
        __syncthreads();  // part[] is rewritten by the next chunk
    }
}

// The same step for rows whose length is a multiple of 16, whose arrays start on 16-byte boundaries and whose keys fit
// in shared memory: a thread owns runs of 16 consecutive columns, so the row costs four dependent trips to memory (the
// neuron's flag; mask and pruning flags, 16 bytes each; the keys, 16-byte loads of only the groups that hold candidates;
// the weights once more for the write-back) instead of one per 256 columns and array, ties are ranked with one block-wide
// prefix count per 4096 columns, and mask and weights go back in whole 16-byte stores.
__global__ void __launch_bounds__(kThreads, 8) finalize_runs_kernel(float* w, uint8_t* mask, const float* grad, const uint8_t* drop, const uint8_t* survives,
                                     int in_f, const Scalars* sc) {
    extern __shared__ __align__(16) unsigned char row_smem[];  // keys[in_f] (4 bytes each), then state[in_f] (1 byte each)
    __shared__ unsigned int hist[256];
    __shared__ RowCut cut;
    __shared__ int kept_count;
    __shared__ unsigned int warp_tot[kThreads / 32];
    const int r = blockIdx.x, t = threadIdx.x, lane = t & 31, wid = t >> 5, n_runs = in_f >> 4;
    float* wr = w + (size_t)r * in_f;
    uint8_t* mr = mask + (size_t)r * in_f;
    const float* gr = grad + (size_t)r * in_f;
    const uint8_t* dr = drop + (size_t)r * in_f;
    if (!survives[r]) {  // ablated now or before: nothing left
        for (int j = t; j < n_runs; j += kThreads) {
            *reinterpret_cast<uint4*>(mr + 16 * j) = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int g = 0; g < 4; ++g) *reinterpret_cast<float4*>(wr + 16 * j + 4 * g) = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        return;
    }
    unsigned int* keys = reinterpret_cast<unsigned int*>(row_smem);
    uint8_t* state = row_smem + (size_t)in_f * 4;  // 1 = kept after step 6, 0 = free
    const int k_new = sc->k_new;
    if (t == 0) kept_count = 0;
    __syncthreads();
    int mine = 0;
    for (int j = t; j < n_runs; j += kThreads) {
        const uint4 m = *reinterpret_cast<const uint4*>(mr + 16 * j), d = *reinterpret_cast<const uint4*>(dr + 16 * j);
        uint4 st;  // a byte per column: 1 where the mask is set and the weight was not pruned in step 6
        st.x = __vcmpne4(m.x, 0u) & __vcmpeq4(d.x, 0u) & 0x01010101u;
        st.y = __vcmpne4(m.y, 0u) & __vcmpeq4(d.y, 0u) & 0x01010101u;
        st.z = __vcmpne4(m.z, 0u) & __vcmpeq4(d.z, 0u) & 0x01010101u;
        st.w = __vcmpne4(m.w, 0u) & __vcmpeq4(d.w, 0u) & 0x01010101u;
        mine += __popc(st.x) + __popc(st.y) + __popc(st.z) + __popc(st.w);
        *reinterpret_cast<uint4*>(state + 16 * j) = st;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mine += __shfl_down_sync(0xffffffffu, mine, off);
    if (lane == 0 && mine) atomicAdd(&kept_count, mine);
    __syncthreads();
    const int kept = kept_count;
    const bool trim = kept > k_new;
    const int m = trim ? kept - k_new : k_new - kept;
    if (m > 0) {
        const float* src = trim ? wr : gr;
        const unsigned int flip = trim ? 0u : 0xFFFFFFFFu;  // regrowing: the complement, so that a larger gradient is a smaller key
        for (int j = t; j < n_runs; j += kThreads) {
            const uint4 st = *reinterpret_cast<const uint4*>(state + 16 * j);
            const unsigned int sw[4] = {st.x, st.y, st.z, st.w};
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                const unsigned int cand = trim ? sw[g] : (sw[g] ^ 0x01010101u);
                uint4 kq = make_uint4(0u, 0u, 0u, 0u);
                if (cand != 0u) {
                    const float4 v = *reinterpret_cast<const float4*>(src + 16 * j + 4 * g);
                    kq.x = (cand & 0x00000001u) ? (mag_bits(v.x) ^ flip) : 0u;
                    kq.y = (cand & 0x00000100u) ? (mag_bits(v.y) ^ flip) : 0u;
                    kq.z = (cand & 0x00010000u) ? (mag_bits(v.z) ^ flip) : 0u;
                    kq.w = (cand & 0x01000000u) ? (mag_bits(v.w) ^ flip) : 0u;
                }
                *reinterpret_cast<uint4*>(keys + 16 * j + 4 * g) = kq;
            }
        }
        __syncthreads();
    }
    // Four columns per thread and step: one 16-byte read of the keys, one 4-byte read of the state bytes.
    row_select(m, [&](unsigned int pre, unsigned int pm, int shift) {
        const unsigned int flip_state = trim ? 0u : 0x01010101u;
        for (int q = t; q < (in_f >> 2); q += kThreads) {
            const unsigned int cand = reinterpret_cast<const unsigned int*>(state)[q] ^ flip_state;
            if (cand == 0u) continue;
            const uint4 kq = reinterpret_cast<const uint4*>(keys)[q];
            if ((cand & 0x00000001u) && (kq.x & pm) == pre) atomicAdd(&hist[(kq.x >> shift) & 255u], 1u);
            if ((cand & 0x00000100u) && (kq.y & pm) == pre) atomicAdd(&hist[(kq.y >> shift) & 255u], 1u);
            if ((cand & 0x00010000u) && (kq.z & pm) == pre) atomicAdd(&hist[(kq.z >> shift) & 255u], 1u);
            if ((cand & 0x01000000u) && (kq.w & pm) == pre) atomicAdd(&hist[(kq.w >> shift) & 255u], 1u);
        }
    }, hist, &cut);
    // Apply in column order, so that ties on the cut key go to the smaller columns: a tie's rank is the ties of the
    // 4096-column chunks before (carried by every thread), of the threads before in this chunk (a prefix count over the
    // block) and of the columns before in the thread's own run.
    const bool any = cut.any != 0;
    const unsigned int cut_key = cut.cut, cut_ties = cut.ties;
    unsigned int carry = 0;
    for (int j0 = 0; j0 < n_runs; j0 += kThreads) {
        const int j = j0 + t;
        const bool have = j < n_runs;
        uint4 st = make_uint4(0u, 0u, 0u, 0u);
        float4 wv[4];
        if (have) {
            st = *reinterpret_cast<const uint4*>(state + 16 * j);
#pragma unroll
            for (int g = 0; g < 4; ++g) wv[g] = *reinterpret_cast<const float4*>(wr + 16 * j + 4 * g);  // in flight during the count
        }
        const unsigned int sw[4] = {st.x, st.y, st.z, st.w};
        unsigned int my_ties = 0;
        if (have && any) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                const uint4 kq = *reinterpret_cast<const uint4*>(keys + 16 * j + 4 * g);
                const unsigned int cand = trim ? sw[g] : (sw[g] ^ 0x01010101u);
                my_ties += ((cand & 0x00000001u) && kq.x == cut_key) + ((cand & 0x00000100u) && kq.y == cut_key) +
                           ((cand & 0x00010000u) && kq.z == cut_key) + ((cand & 0x01000000u) && kq.w == cut_key);
            }
        }
        unsigned int incl = my_ties;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned int up = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += up;
        }
        if (lane == 31) warp_tot[wid] = incl;
        __syncthreads();
        unsigned int rank = carry + incl - my_ties, in_chunk = 0;
#pragma unroll
        for (int i = 0; i < kThreads / 32; ++i) {
            const unsigned int p = warp_tot[i];
            rank += i < wid ? p : 0u;
            in_chunk += p;
        }
        if (have) {
            unsigned int mo[4];
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                uint4 kq = make_uint4(0u, 0u, 0u, 0u);
                if (any) kq = *reinterpret_cast<const uint4*>(keys + 16 * j + 4 * g);
                const unsigned int kk[4] = {kq.x, kq.y, kq.z, kq.w};
                float we[4] = {wv[g].x, wv[g].y, wv[g].z, wv[g].w};
                mo[g] = 0u;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const bool is_kept = ((sw[g] >> (8 * e)) & 1u) != 0u;
                    const bool candidate = trim ? is_kept : !is_kept;
                    const bool tie = any && candidate && kk[e] == cut_key;
                    bool selected = any && candidate && kk[e] < cut_key;
                    if (tie) selected = rank++ < cut_ties;
                    const bool on = trim ? (is_kept && !selected) : (is_kept || selected);
                    if (!on || !is_kept) we[e] = 0.0f;  // pruned, trimmed, free, or grown (starts at 0); a survivor keeps its value
                    mo[g] |= (on ? 1u : 0u) << (8 * e);
                }
                *reinterpret_cast<float4*>(wr + 16 * j + 4 * g) = make_float4(we[0], we[1], we[2], we[3]);
            }
            *reinterpret_cast<uint4*>(mr + 16 * j) = make_uint4(mo[0], mo[1], mo[2], mo[3]);
        }
        carry += in_chunk;
        __syncthreads();  // warp_tot[] is rewritten by the next chunk
    }
}

size_t align_up(size_t v) { return (v + 255) & ~(size_t)255; }

struct Workspace {
    int* row_count;
    int* salient;
    uint8_t* survives;
    uint8_t* drop;
    uint8_t* grow_top;
    unsigned int* chunk_ties;
    uint2* list;            // 2 x list_capacity(n) (key, position) pairs
    SelectState* state;
    Scalars* scalars;
    size_t bytes;
};

Workspace carve(void* base, int out_f, int in_f) {
    const size_t n = (size_t)out_f * in_f, chunks = (n + kChunk - 1) / kChunk;
    size_t off = 0;
    auto take = [&](size_t b) {
        const size_t at = off;
        off += align_up(b);
        return static_cast<char*>(base) + at;
    };
    Workspace w{};
    w.row_count = reinterpret_cast<int*>(take((size_t)out_f * 4));
    w.salient = reinterpret_cast<int*>(take((size_t)out_f * 4));
    w.survives = reinterpret_cast<uint8_t*>(take((size_t)out_f));
    w.drop = reinterpret_cast<uint8_t*>(take(n));
    w.grow_top = reinterpret_cast<uint8_t*>(take(n));
    w.chunk_ties = reinterpret_cast<unsigned int*>(take(2 * chunks * 4));
    w.list = reinterpret_cast<uint2*>(take(2 * (size_t)list_capacity((long long)n) * sizeof(uint2)));
    w.state = reinterpret_cast<SelectState*>(take(2 * sizeof(SelectState)));
    w.scalars = reinterpret_cast<Scalars*>(take(sizeof(Scalars)));
    w.bytes = off;
    return w;
}

// Step 3's two selections over the whole layer (the first is also step 6's pruning set), in shared sweeps.
bool layer_select_both(const float* w, const uint8_t* mask, const float* grad, const Workspace& ws, int out_f, int in_f,
                       long long n, cudaStream_t st) {
    const int chunks = (int)((n + kChunk - 1) / kChunk);
    const int hist_blocks = out_f < 1184 ? out_f : 1184;  // whole rows per block, 8 CTAs per SM at most
    for (int pass = 0; pass < 4; ++pass) {
        if (pass < 3)
            hist_kernel<false><<<hist_blocks, kThreads, 0, st>>>(w, mask, grad, ws.row_count, out_f, in_f, pass, ws.state, ws.list,
                                                                 list_capacity(n));
        else
            hist_kernel<true><<<hist_blocks, kThreads, 0, st>>>(w, mask, grad, ws.row_count, out_f, in_f, pass, ws.state, ws.list,
                                                                list_capacity(n));
    }
    // 16-byte loads and stores of a thread's run of 16 positions: the run must lie inside one row, and the arrays (the
    // workspace's flag arrays are 256-byte aligned) must start on 16-byte boundaries.
    const bool vec_ok = (in_f % 16) == 0 && ((reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(grad) |
                                               reinterpret_cast<uintptr_t>(mask)) & 15u) == 0;
    tie_count_kernel<<<chunks, kThreads, 0, st>>>(w, mask, grad, ws.row_count, in_f, n, ws.state, ws.chunk_ties, chunks, vec_ok);
    chunk_scan_kernel<<<2, kThreads, 0, st>>>(ws.chunk_ties, chunks, ws.state);
    mark_kernel<<<chunks, kThreads, 0, st>>>(w, mask, grad, ws.row_count, in_f, n, ws.state, ws.chunk_ties, chunks, ws.drop,
                                             ws.grow_top, vec_ok);
    return cudaGetLastError() == cudaSuccess;
}

// ---- cfi_pack_device: the condensed arrays straight from device-resident w and mask -------------------------------

// Single block: rank of every non-empty row among the non-empty rows, their number, the common fan-in, and whether the
// fan-in really is common.  info = {n_active, k, constant (1/0)}.
__global__ void pack_rows_kernel(const int* row_count, int out_f, int* row_rank, int* info) {
    __shared__ unsigned int part[kThreads];
    __shared__ unsigned int carry;
    __shared__ int k_min, k_max;
    if (threadIdx.x == 0) carry = 0, k_min = 0x7fffffff, k_max = 0;
    __syncthreads();
    for (int r0 = 0; r0 < out_f; r0 += kThreads) {
        const int r = r0 + threadIdx.x;
        const int cnt = r < out_f ? row_count[r] : 0;
        const unsigned int live = cnt > 0 ? 1u : 0u;
        if (live) atomicMin(&k_min, cnt), atomicMax(&k_max, cnt);
        part[threadIdx.x] = live;
        __syncthreads();
        for (int off = 1; off < kThreads; off <<= 1) {
            const unsigned int add = threadIdx.x >= off ? part[threadIdx.x - off] : 0u;
            __syncthreads();
            part[threadIdx.x] += add;
            __syncthreads();
        }
        if (r < out_f) row_rank[r] = live ? (int)(carry + part[threadIdx.x] - 1) : -1;
        __syncthreads();
        if (threadIdx.x == kThreads - 1) carry += part[kThreads - 1];
        __syncthreads();
    }
    if (threadIdx.x == 0) info[0] = (int)carry, info[1] = k_max, info[2] = (carry == 0 || k_min == k_max) ? 1 : 0;
}

// One block per row: its kept entries in increasing column order to values / indices of its rank.
__global__ void pack_fill_kernel(const float* w, const uint8_t* mask, const int* row_rank, int in_f, int k, float* values,
                                 int32_t* indices, int32_t* active_rows) {
    __shared__ unsigned int part[kThreads];
    __shared__ unsigned int carry;
    const int r = blockIdx.x, rank = row_rank[r];
    if (rank < 0) return;
    if (threadIdx.x == 0) carry = 0, active_rows[rank] = r;
    __syncthreads();
    const float* wr = w + (size_t)r * in_f;
    const uint8_t* mr = mask + (size_t)r * in_f;
    for (int c0 = 0; c0 < in_f; c0 += kThreads) {
        const int c = c0 + threadIdx.x;
        const unsigned int kept = (c < in_f && mr[c]) ? 1u : 0u;
        part[threadIdx.x] = kept;
        __syncthreads();
        for (int off = 1; off < kThreads; off <<= 1) {
            const unsigned int add = threadIdx.x >= off ? part[threadIdx.x - off] : 0u;
            __syncthreads();
            part[threadIdx.x] += add;
            __syncthreads();
        }
        if (kept) {
            const size_t at = (size_t)rank * k + carry + part[threadIdx.x] - 1;
            values[at] = wr[c];
            indices[at] = c;
        }
        __syncthreads();
        if (threadIdx.x == kThreads - 1) carry += part[kThreads - 1];
        __syncthreads();
    }
}

}  // namespace

extern "C" cfi_status_t cfi_srigl_workspace_bytes(int32_t out_features, int32_t in_features, size_t* bytes) {
    if (!bytes) return CFI_ERR_NULL;
    if (out_features < 1 || in_features < 1 || (int64_t)out_features * in_features > ((int64_t)1 << 31)) return CFI_ERR_SHAPE;
    *bytes = carve(nullptr, out_features, in_features).bytes;
    return CFI_OK;
}

extern "C" cfi_status_t cfi_srigl_update(float* w, uint8_t* mask, const float* grad, int32_t out_features, int32_t in_features,
                                         int64_t K, float gamma_sal, void* workspace, size_t workspace_bytes, int32_t* k_new,
                                         int32_t* n_active_new, cfi_stream_t stream) {
    if (!w || !mask || !grad || !workspace || !k_new || !n_active_new) return CFI_ERR_NULL;
    if (out_features < 1 || in_features < 1 || (int64_t)out_features * in_features > ((int64_t)1 << 31) || !(gamma_sal >= 0.0f))
        return CFI_ERR_SHAPE;
    if (((uintptr_t)workspace & 255) != 0) return CFI_ERR_ALIGNMENT;
    const Workspace ws = carve(workspace, out_features, in_features);
    if (workspace_bytes < ws.bytes) return CFI_ERR_BUFFER_TOO_SMALL;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const long long n = (long long)out_features * in_features;
    row_count_kernel<<<out_features, kThreads, 0, st>>>(mask, out_features, in_features, ws.row_count);
    setup_kernel<<<1, kThreads, 0, st>>>(ws.row_count, out_features, in_features, (long long)K, ws.scalars, ws.state);
    if (!layer_select_both(w, mask, grad, ws, out_features, in_features, n, st)) return CFI_ERR_CUDA;
    salient_kernel<<<out_features, kThreads, 0, st>>>(mask, ws.drop, ws.grow_top, in_features, ws.salient);
    ablate_kernel<<<1, kThreads, 0, st>>>(ws.row_count, ws.salient, out_features, in_features, gamma_sal, ws.scalars, ws.survives);
    const size_t row_bytes = (size_t)in_features * 5;  // keys and one state byte per column
    const bool runs_ok = (in_features % 16) == 0 && ((reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(grad) |
                                                         reinterpret_cast<uintptr_t>(mask)) & 15u) == 0;
    if (row_bytes <= 40 * 1024 && runs_ok && in_features >= 2048)  // shorter rows leave most of a block's threads without a run
        finalize_runs_kernel<<<out_features, kThreads, row_bytes, st>>>(w, mask, grad, ws.drop, ws.survives, in_features, ws.scalars);
    else if (row_bytes <= 40 * 1024)
        finalize_kernel<true><<<out_features, kThreads, row_bytes, st>>>(w, mask, grad, ws.drop, ws.survives, in_features, ws.scalars);
    else
        finalize_kernel<false><<<out_features, kThreads, 0, st>>>(w, mask, grad, ws.drop, ws.survives, in_features, ws.scalars);
    Scalars host{};
    if (cudaGetLastError() != cudaSuccess ||
        cudaMemcpyAsync(&host, ws.scalars, sizeof(host), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return CFI_ERR_CUDA;
    }
    *k_new = host.k_new;
    *n_active_new = host.live_after;
    return CFI_OK;
}

extern "C" cfi_status_t cfi_pack_device(const float* w_dense, const uint8_t* mask, int32_t out_features, int32_t in_features,
                                        void* workspace, size_t workspace_bytes, int32_t* k, int32_t* n_active, float* values,
                                        int32_t* indices, int32_t* active_rows, cfi_stream_t stream) {
    if (!w_dense || !mask || !workspace || !k || !n_active) return CFI_ERR_NULL;
    if (out_features < 1 || in_features < 1 || (int64_t)out_features * in_features > ((int64_t)1 << 31)) return CFI_ERR_SHAPE;
    const bool fill = values || indices || active_rows;
    if (fill && !(values && indices && active_rows)) return CFI_ERR_NULL;
    if (((uintptr_t)workspace & 255) != 0) return CFI_ERR_ALIGNMENT;
    if (workspace_bytes < (size_t)out_features * 8 + 256) return CFI_ERR_BUFFER_TOO_SMALL;
    int* row_count = static_cast<int*>(workspace);
    int* row_rank = row_count + out_features;
    int* info = row_rank + out_features;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    row_count_kernel<<<out_features, kThreads, 0, st>>>(mask, out_features, in_features, row_count);
    pack_rows_kernel<<<1, kThreads, 0, st>>>(row_count, out_features, row_rank, info);
    int host[3] = {0, 0, 0};
    if (cudaGetLastError() != cudaSuccess || cudaMemcpyAsync(host, info, sizeof(host), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return CFI_ERR_CUDA;
    }
    if (!host[2]) return CFI_ERR_NOT_CONSTANT_FAN_IN;
    *n_active = host[0];
    *k = host[0] ? host[1] : 0;
    if (!fill || host[0] == 0) return CFI_OK;
    pack_fill_kernel<<<out_features, kThreads, 0, st>>>(w_dense, mask, row_rank, in_features, host[1], values, indices, active_rows);
    if (cudaGetLastError() != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return CFI_ERR_CUDA;
    }
    return CFI_OK;
}
