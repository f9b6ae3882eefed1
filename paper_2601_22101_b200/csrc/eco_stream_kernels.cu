// Streaming kernels of the ECO step for sm_100a: persistent CTAs fed by the TMA
// engine.
//
// One CTA = 1 producer warp + 8 consumer warps, two (Adam) or three (momentum SGD) CTAs per SM.  The parameter
// set is cut into units of 32 rows of 128 elements (4096 parameters), handed out to
// the CTAs by a device-wide ticket counter.  For every unit the producer issues one
// bulk asynchronous copy (cp.async.bulk, global -> shared, completion counted
// on an mbarrier) per input stream -- codes, bf16 gradient, m and, for Adam, v
// -- into a ring of shared-memory stages, and stages the unit's old scales and
// a small header next to them.  Consumer warps wait for the stage, pull their 4
// rows out of shared memory with conflict-free 16-byte reads, hand the stage
// back, and do all arithmetic from registers; results go straight to global
// memory with coalesced 16-byte stores.  Global loads therefore cost no issue
// slots and no registers, and the bytes in flight per SM are set by the ring
// depth (tens of KB), not by occupancy.
//
// Every wait on an mbarrier is bounded: after ~2 s worth of clock cycles the
// waiter records a code in the context's status word and leaves; the producer
// first waits (bounded again) for the copies it has in flight.
#include "eco_device.cuh"
#include "eco_index.h"
#include "eco_launch.h"

namespace eco {

constexpr int kConsumerWarps = 8;
constexpr int kStreamThreads = (kConsumerWarps + 1) * 32;
constexpr int kUnitRows = kConsumerWarps * 4;      // rows of 128 elements per unit
constexpr long long kWaitLimitCycles = 4000000000LL;
constexpr int kInterleave = 8;                     // regions of a block-scale launch walked concurrently

// What the producer tells the consumers about a unit.
struct StageHeader {
    uint8_t* w;
    void* scale;
    float* m;
    float* v;
    uint64_t row0;        // first row of the unit inside its tensor
    uint32_t nrows;       // rows present (the last unit of a tensor may be short)
    uint32_t tensor_id;
    uint32_t slot;
    float s_old;          // per-tensor modes
    float s_new, inv_new; // per-tensor pass 2
    uint32_t seg_per_row; // per-row mode: 128-element rows per matrix row (R)
    uint32_t div_magic;   // per-row mode: floor(65536 / R) + 1, so that (x * div_magic) >> 16 == x / R for x < 2048
    uint32_t n_mrows;     // per-row mode: matrix rows in the unit
    uint32_t pass;        // wave kernel: what this publication is (WAVE_*)
    uint64_t mrow0;       // per-row mode: first matrix row of the unit
    uint64_t index_base;  // element index of the tensor's first element inside the full (unsharded) tensor
    float* e;             // optional error buffer of the tensor (NULL: none)
    uint32_t barrier_target;   // wave kernel: non-zero = wait until the grid counter reaches this before going on
    uint32_t first_of_tensor;  // wave kernel: this unit is the first of its tensor (its consumers store the new scale)
};
static_assert(sizeof(StageHeader) <= 128, "header must fit its slot");

// Resident CTAs per SM a kernel instantiation is compiled for (register budget 65536 / (288 * n)).
template <int OPT, bool ERR>
__host__ __device__ constexpr int stream_ctas_per_sm() { return (OPT == OPT_SGDM && !ERR) ? 3 : 2; }

template <int FMT, int OPT>
struct StageLayout {
    static constexpr int kCodeRow = FMT == FMT_INT4 ? 64 : 128;  // bytes of codes per row
    static constexpr int kHeader = 0;
    static constexpr int kScales = 128;                          // up to 4 floats per row (blocks of 32 elements)
    static constexpr int kCodes = kScales + kUnitRows * 16;
    static constexpr int kGrad = kCodes + kUnitRows * kCodeRow;
    static constexpr int kM = kGrad + kUnitRows * 256;
    static constexpr int kV = kM + kUnitRows * 512;
    static constexpr int kBytes = kV + (OPT == OPT_ADAM ? kUnitRows * 512 : 0);
    static constexpr int kStages = 2;                            // x 2 (Adam) or 3 (SGDM) resident CTAs per SM
    static constexpr int kBarriers = 512;                        // 2 * kStages + 2 mbarriers, padded to 128; then the
                                                                 // per-row exchange: 32 maxima, 32 scales, 32 inverses
    static constexpr int kRowBars = 64;                          // two mbarriers of the per-row exchange
    static constexpr int kClusterBars = 96;                      // per-row mode in a cluster: the two mbarriers the peers arrive on
    static constexpr int kExchange = 128;                        // the exchange arrays (in a cluster: 2 x 4 x 8 partial row maxima)
    static_assert(2 * kStages * 8 <= kRowBars, "the stage barriers end before the exchange barriers");
    static_assert(kExchange + 2 * 4 * kConsumerWarps * 4 <= kBarriers && kExchange + 96 * 4 <= kBarriers, "exchange arrays fit");
    static constexpr int kSmem = kBarriers + kStages * kBytes;
    static_assert(kBytes % 128 == 0, "stages stay 128-byte aligned");
};

// ---- mbarrier / bulk-copy primitives ----------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.shared::cta.b64 st, [%0]; }" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait; on expiry records `code` and returns false.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t* status, uint32_t code,
                                          long long limit_cycles = kWaitLimitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > limit_cycles) {
            atomicExch(status, code);
            return false;
        }
    }
    return true;
}
// Plain (single-CTA) bulk copy global -> shared, completion on an mbarrier of this CTA.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// The same with an L2 eviction-priority hint (a policy made by createpolicy) for this copy's lines.
__device__ __forceinline__ void bulk_load_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
// 16- and 4/2-byte stores whose lines L2 may drop first (results that are not read again within the step).
__device__ __forceinline__ void store_f4_first(float* p, float a, float b, float c, float d, uint64_t policy) {
    asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d), "l"(policy) : "memory");
}
__device__ __forceinline__ void store_u32_first(void* p, uint32_t v, uint64_t policy) {
    asm volatile("st.global.L2::cache_hint.u32 [%0], %1, %2;" ::"l"(p), "r"(v), "l"(policy) : "memory");
}
__device__ __forceinline__ void store_u16_first(void* p, uint32_t v, uint64_t policy) {
    asm volatile("st.global.L2::cache_hint.u16 [%0], %1, %2;" ::"l"(p), "h"(static_cast<uint16_t>(v)), "l"(policy) : "memory");
}

// ---- thread-block cluster primitives (per-row scales on rows longer than one unit) ----
__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_size() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r)); return r; }
// Address of the same shared-memory location in CTA `rank` of this cluster.
__device__ __forceinline__ uint32_t peer_addr(uint32_t local, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ void peer_store_f32(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
// Arrival on a peer's mbarrier; release at cluster scope orders this thread's earlier peer stores before it.
__device__ __forceinline__ void peer_mbar_arrive(uint32_t addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
// One binary32 value into a peer's shared memory, counted as 4 bytes of the transaction the peer's mbarrier expects:
// the barrier's wait then makes the value visible, no fence by the sender.
__device__ __forceinline__ void peer_store_async_f32(uint32_t addr, float v, uint32_t bar_addr) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
                 ::"r"(addr), "r"(__float_as_uint(v)), "r"(bar_addr) : "memory");
}
// Bounded wait on an own mbarrier that peers arrive on (acquire at cluster scope).
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, uint32_t* status, uint32_t code) {
    const long long t0 = clock64();
    for (;;) {
        uint32_t ok;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if (clock64() - t0 > kWaitLimitCycles) {
            atomicExch(status, code);
            return false;
        }
    }
}

// max |x| over the 32 lanes in one instruction (sm_100a warp reduction on binary32; NaN operands are
// ignored, as by fmaxf).  Every lane receives the result.  The final maximum with zero makes a warp whose
// operands are ALL NaN return 0 (a block of nothing but NaN has no maximum: it takes the scale of an all-zero block).
__device__ __forceinline__ float warp_amax(float x) {
    float r;
    asm volatile("redux.sync.max.abs.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(x));
    return fmaxf(r, 0.0f);
}

__device__ __forceinline__ uint32_t units_of(const TensorDesc& T) {
    return static_cast<uint32_t>((T.n_blocks + kUnitRows - 1) / kUnitRows);
}

// One unit (up to 32 rows of 128 elements) by the 8 consumer warps: warp w owns rows 4w..4w+3, lane l
// elements 4l..4l+3 of each.  FULL: all 32 rows are present (every unit but the last of a tensor).
// TS: the scales of the per-tensor modes (old scale for the dequantization; new scale and its inverse for pass 2).
struct TensorScales { float s_old, s_new, inv_new; };
// Per-row mode inside a thread-block cluster: this CTA's rank, the cluster's size (1 = no cluster), the shared-memory
// addresses of the exchange slots and barriers, and the phase parity of the barrier this unit uses.
struct ClusterInfo {
    uint32_t rank, size, peer_max, bars, phase;
    const float* peer_max_ptr;
};
// HINT: stores carry an evict-first hint (`store_policy`); false = plain stores.
template <int FMT, int OPT, int RND, int MODE, bool FULL, bool ERR, int NS = 4, bool HINT = false>
__device__ __forceinline__ bool consume_unit(const StepParams& P, const int scale_kind, const uint8_t* st,
                                             const StageHeader* h, const uint32_t empty_bar, const int warp,
                                             const int lane, uint32_t* scratch_amax, uint32_t& cur_slot,
                                             float& run_max, float* xchg, const uint32_t row_bars,
                                             const uint32_t row_parity, uint32_t* status,
                                             const TensorScales ts = TensorScales{1.0f, 1.0f, 1.0f},
                                             const uint64_t store_policy = 0,
                                             const ClusterInfo cl = ClusterInfo{0u, 1u, 0u, 0u, 0u, nullptr}) {
    using SL = StageLayout<FMT, OPT>;
    // Row (of 128 elements) behind slot k of this warp.  Per-row mode deals the rows round-robin (warp, warp + 8, ...)
    // so that a unit of fewer than 32 rows leaves every warp with 3 or 4 rows instead of some with none; NS is the
    // number of slots this instantiation carries (with FULL: all of them present).
    static_assert(NS == 4 || MODE == MODE_ROW, "only the per-row mode runs with fewer slots");
    constexpr int kRowStep = MODE == MODE_ROW ? kConsumerWarps : 1;
    const int r = MODE == MODE_ROW ? warp : warp * 4;
    const int nrows = static_cast<int>(h->nrows);
    const uint64_t i_first = (h->row0 + r) * 128 + lane * 4;      // element index of (slot 0, this lane)
    float* const vp = h->v;

    Lane4<OPT> L[NS];
    float amax[NS];
    {
        float th[NS][4], g[NS][4], m[NS][4], v[NS][4], vt[NS][4];
#pragma unroll
        for (int k = 0; k < NS; ++k) {
            const int row = r + k * kRowStep;
            const bool valid = FULL || row < nrows;
            uint32_t codes = 0;
            float s_old = 1.0f;
#pragma unroll
            // rows that are not present (short units) carry harmless values: their results are never stored, and
            // ones keep the thread on the straight-line square root / division path (zeros would not)
            for (int e = 0; e < 4; ++e) { g[k][e] = 0.f; m[k][e] = 1.f; v[k][e] = 1.f; }
            if (valid) {
                if (FMT != FMT_INT4) codes = *reinterpret_cast<const uint32_t*>(st + SL::kCodes + row * 128 + lane * 4);
                else codes = *reinterpret_cast<const uint16_t*>(st + SL::kCodes + row * 64 + lane * 2);
                const uint2 gr = *reinterpret_cast<const uint2*>(st + SL::kGrad + row * 256 + lane * 8);
                g[k][0] = __uint_as_float(gr.x << 16); g[k][1] = __uint_as_float(gr.x & 0xFFFF0000u);
                g[k][2] = __uint_as_float(gr.y << 16); g[k][3] = __uint_as_float(gr.y & 0xFFFF0000u);
                const float4 mr = *reinterpret_cast<const float4*>(st + SL::kM + row * 512 + lane * 16);
                m[k][0] = mr.x; m[k][1] = mr.y; m[k][2] = mr.z; m[k][3] = mr.w;
                if (OPT == OPT_ADAM) {
                    const float4 vr = *reinterpret_cast<const float4*>(st + SL::kV + row * 512 + lane * 16);
                    v[k][0] = vr.x; v[k][1] = vr.y; v[k][2] = vr.z; v[k][3] = vr.w;
                }
                if (MODE == MODE_BLOCK) s_old = reinterpret_cast<const float*>(st + SL::kScales)[row];
                else if (MODE == MODE_BLOCK32) s_old = reinterpret_cast<const float*>(st + SL::kScales)[row * 4 + (lane >> 3)];
                else if (MODE == MODE_ROW) s_old = reinterpret_cast<const float*>(st + SL::kScales)[(row * h->div_magic) >> 16];
                else s_old = ts.s_old;
            }
            float val[4];
            unpack4<FMT>(codes, val);
#pragma unroll
            for (int p = 0; p < 4; p += 2) {
                const float2 t = mul2(make_float2(val[p], val[p + 1]), dup2(s_old));
                th[k][p] = t.x; th[k][p + 1] = t.y;
            }
        }
        optim_rows<OPT, NS>(P, th, g, m, v, L, vt);
#pragma unroll
        for (int k = 0; k < NS; ++k) {
            const bool valid = FULL || r + k * kRowStep < nrows;
            amax[k] = 0.0f;
            if (valid) amax[k] = fmaxf(fmaxf(fabsf(L[k].tht[0]), fabsf(L[k].tht[1])), fmaxf(fabsf(L[k].tht[2]), fabsf(L[k].tht[3])));
            if (OPT == OPT_ADAM && MODE != MODE_TENSOR_AMAX && valid) {
                if (HINT) store_f4_first(vp + i_first + k * (kRowStep * 128), vt[k][0], vt[k][1], vt[k][2], vt[k][3], store_policy);
                else *reinterpret_cast<float4*>(vp + i_first + k * (kRowStep * 128)) = make_float4(vt[k][0], vt[k][1], vt[k][2], vt[k][3]);
            }
        }
    }
    // everything needed later is read before the stage is handed back
    uint8_t* const wp = h->w;
    float* const mp = h->m;
    void* const sp = h->scale;
    const uint64_t row0 = h->row0;
    const uint32_t tensor_id = h->tensor_id, slot = h->slot;
    const float s_new = ts.s_new, inv_new = ts.inv_new;
    const uint32_t seg_per_row = h->seg_per_row, div_magic = h->div_magic, n_mrows = h->n_mrows;
    const uint64_t mrow0 = h->mrow0;
    // Per-lane bases, formed once per unit; the slots of a lane then differ by compile-time constants only
    // (row step * 128 elements: a multiple of 4, so the shifts below commute with adding it).
    uint8_t* const w_lane = wp + (FMT != FMT_INT4 ? i_first : (i_first >> 1));
    float* const m_lane = mp + i_first;
    float* const e_lane = ERR ? h->e + i_first : nullptr;
    const uint32_t ctr_lane = static_cast<uint32_t>((i_first + h->index_base) >> 2);   // Philox counter of slot 0
    // (INT4 + momentum SGD with block scales hands the stage back after the row maxima instead: three CTAs per SM
    // keep the copy engine busy anyway, and the compiler then fits the lane's state into its 72 registers)
    constexpr bool kLateRelease = MODE == MODE_BLOCK && OPT == OPT_SGDM && FMT == FMT_INT4;
    if (!kLateRelease) {
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar);      // the stage may be refilled
    }

    if (MODE == MODE_TENSOR_AMAX) {
        if (slot != cur_slot) {
            if (cur_slot != 0xFFFFFFFFu) {
                const float z = warp_amax(run_max);
                if (lane == 0) atomicMax(scratch_amax + cur_slot, __float_as_uint(z));
            }
            cur_slot = slot;
            run_max = 0.0f;
        }
#pragma unroll
        for (int k = 0; k < NS; ++k) run_max = fmaxf(run_max, amax[k]);
        return true;
    }

    float s_k[NS], inv_k[NS];
    if (MODE == MODE_BLOCK) {
        // row maxima: one warp reduction per row; lane group g = lane / 8 then derives the scale of row g
        // and the four scales are broadcast from lanes 0, 8, 16, 24
        float rmax[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) rmax[k] = warp_amax(amax[k]);
        const int g8 = lane >> 3;
        const float my_amax = g8 == 0 ? rmax[0] : (g8 == 1 ? rmax[1] : (g8 == 2 ? rmax[2] : rmax[3]));
        float s_mine, inv_mine;
        uint32_t bits_mine;
        make_scale_div<FMT>(my_amax, scale_kind == SCALE_KIND_BF16, s_mine, inv_mine, bits_mine);
        if ((lane & 7) == 0 && (FULL || r + g8 < nrows))
            store_scale(sp, row0 + r + g8, scale_kind, s_mine, bits_mine);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            s_k[k] = __shfl_sync(0xFFFFFFFFu, s_mine, 8 * k);
            inv_k[k] = __shfl_sync(0xFFFFFFFFu, inv_mine, 8 * k);
        }
        if (kLateRelease) {
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar);
        }
    } else if (MODE == MODE_BLOCK32) {
        // Four scale blocks of 32 elements per row, 8 lanes each: 16 maxima per warp.  Three butterfly stages inside
        // each group of 8 lanes, halving the number of rows a lane carries at each: afterwards lane l holds the
        // maximum of row (l >> 1) & 3 over its group.  It derives that one scale; the four scales a lane needs come
        // back from lanes 0, 2, 4, 6 of its group.
        const bool b2 = lane & 4, b1 = lane & 2;
        const float x = fmaxf(b2 ? amax[2] : amax[0], __shfl_xor_sync(0xFFFFFFFFu, b2 ? amax[0] : amax[2], 4));
        const float y = fmaxf(b2 ? amax[3] : amax[1], __shfl_xor_sync(0xFFFFFFFFu, b2 ? amax[1] : amax[3], 4));
        float z = fmaxf(b1 ? y : x, __shfl_xor_sync(0xFFFFFFFFu, b1 ? x : y, 2));
        z = fmaxf(fmaxf(z, __shfl_xor_sync(0xFFFFFFFFu, z, 1)), 0.0f);     // (an all-NaN block: 0, like warp_amax)
        const int rr = (lane >> 1) & 3, g8 = lane >> 3;
        float s_mine, inv_mine;
        uint32_t bits_mine;
        make_scale_pow2<FMT>(z, s_mine, inv_mine, bits_mine);
        if ((lane & 1) == 0 && (FULL || r + rr < nrows))
            static_cast<uint8_t*>(sp)[(row0 + r + rr) * 4 + g8] = static_cast<uint8_t>(bits_mine);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            s_k[k] = __shfl_sync(0xFFFFFFFFu, s_mine, (lane & 24) + 2 * k);
            inv_k[k] = __shfl_sync(0xFFFFFFFFu, inv_mine, (lane & 24) + 2 * k);
        }
    } else if (MODE == MODE_ROW && cl.size > 1) {
        // A matrix row longer than one unit: this unit is the slice of ONE matrix row that this CTA of the cluster
        // holds.  Every warp reduces its segments to one partial maximum and hands it to every CTA of the cluster --
        // lane r sends it into CTA r's slot (its own included) with an asynchronous store that counts 4 bytes on CTA r's
        // mbarrier -- then waits, bounded, on its own CTA's barrier (8 arrivals of its own warps, each announcing the
        // 4 x size bytes sent for it), reduces the 8 x size partials and derives the scale itself: one hop across the
        // cluster, no fence, no meeting of the warps before or after it.  Slots and barriers alternate with the
        // unit's parity, so a CTA that is a unit ahead cannot disturb one still reading (bytes that arrive before the
        // announcement just run the barrier's transaction count negative for a while).
        float z = amax[0];
#pragma unroll
        for (int k = 1; k < NS; ++k) z = fmaxf(z, amax[k]);
        z = warp_amax(z);
        const uint32_t slot = cl.peer_max + ((row_parity * 4u + cl.rank) * kConsumerWarps + static_cast<uint32_t>(warp)) * 4u;
        const uint32_t bar = cl.bars + row_parity * 8u;
        // (this warp's arrival on its own barrier announces the 4 bytes each CTA of the cluster sends for it)
        if (lane == 0) mbar_arrive_expect_tx(bar, cl.size * 4u);
        if (static_cast<uint32_t>(lane) < cl.size) peer_store_async_f32(peer_addr(slot, lane), z, peer_addr(bar, lane));
        if (!mbar_wait_cluster(bar, cl.phase, status, 9u)) return false;
        const float* pm = cl.peer_max_ptr + row_parity * (4u * kConsumerWarps);
        const float a = warp_amax(static_cast<uint32_t>(lane) < cl.size * kConsumerWarps ? pm[lane] : 0.0f);
        float s_j, inv_j;
        uint32_t bits_j;
        make_scale_div<FMT>(a, scale_kind == SCALE_KIND_BF16, s_j, inv_j, bits_j);
        if (cl.rank == 0u && warp == 0 && lane == 0) store_scale(sp, mrow0, scale_kind, s_j, bits_j);
#pragma unroll
        for (int k = 0; k < NS; ++k) { s_k[k] = s_j; inv_k[k] = inv_j; }
    } else if (MODE == MODE_ROW) {
        // One scale per matrix row = seg_per_row consecutive 128-element rows, which belong to several warps.
        // Every warp posts the maxima of its 4 rows in shared memory; after the first barrier warp w reduces
        // matrix rows w, w + 8, ... and posts scale and inverse; after the second barrier all read theirs.
        // Both barriers are mbarriers with bounded waits (8 arrivals, one per consumer warp).
        float* xmax = xchg;
        float* xs = xchg + 32;
        float* xinv = xchg + 64;
#pragma unroll
        for (int k = 0; k < NS; ++k) {
            const float z = warp_amax(amax[k]);
            if (lane == 0) xmax[r + k * kRowStep] = z;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(row_bars);
        if (!mbar_wait(row_bars, row_parity, status, 4u)) return false;
        for (uint32_t j = static_cast<uint32_t>(warp); j < n_mrows; j += kConsumerWarps) {
            const float x = static_cast<uint32_t>(lane) < seg_per_row ? xmax[j * seg_per_row + lane] : 0.0f;
            const float a = warp_amax(x);
            float s_j, inv_j;
            uint32_t bits_j;
            make_scale_div<FMT>(a, scale_kind == SCALE_KIND_BF16, s_j, inv_j, bits_j);
            if (lane == 0) {
                xs[j] = s_j;
                xinv[j] = inv_j;
                store_scale(sp, mrow0 + j, scale_kind, s_j, bits_j);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(row_bars + 8);
        if (!mbar_wait(row_bars + 8, row_parity, status, 5u)) return false;
#pragma unroll
        for (int k = 0; k < NS; ++k) {
            const uint32_t j = (static_cast<uint32_t>(r + k * kRowStep) * div_magic) >> 16;
            const bool valid = FULL || r + k * kRowStep < nrows;
            s_k[k] = valid ? xs[j] : 1.0f;
            inv_k[k] = valid ? xinv[j] : 1.0f;
        }
    } else {
#pragma unroll
        for (int k = 0; k < NS; ++k) { s_k[k] = s_new; inv_k[k] = inv_new; }
    }
#pragma unroll
    for (int k = 0; k < NS; ++k) {
        if (!FULL && r + k * kRowStep >= nrows) continue;
        constexpr int kSlotElems = kRowStep * 128;                   // elements between two slots of a lane
        uint32_t word[4] = {0u, 0u, 0u, 0u};
        if (RND == RND_SR) {
            const uint4 rw = philox4x32_10(ctr_lane + static_cast<uint32_t>(k * (kSlotElems / 4)), tensor_id, P.step_lo, P.step_hi, P);
            word[0] = rw.x; word[1] = rw.y; word[2] = rw.z; word[3] = rw.w;
        }
        float mh[4], e_prev[4] = {0.0f, 0.0f, 0.0f, 0.0f}, e_out[4];
        if (ERR && P.inject == 2) {
            const float4 er = *reinterpret_cast<const float4*>(e_lane + k * kSlotElems);
            e_prev[0] = er.x; e_prev[1] = er.y; e_prev[2] = er.z; e_prev[3] = er.w;
        }
        // power-of-two scales make q s exact; INT4 kernels ask the step parameters (bf16 scales do too); the 8-bit
        // float kernels with f32 / bf16 scales take the two-operation form without asking
        constexpr int kExact = MODE == MODE_BLOCK32 ? 1 : (FMT == FMT_INT4 ? -1 : 0);
        const uint32_t codes = back4<FMT, OPT, RND, ERR, kExact>(P, word, s_k[k], inv_k[k], L[k], mh, e_prev, e_out);
        if (HINT) {
            if (FMT != FMT_INT4) store_u32_first(w_lane + k * kSlotElems, codes, store_policy);
            else store_u16_first(w_lane + k * (kSlotElems / 2), codes, store_policy);
            store_f4_first(m_lane + k * kSlotElems, mh[0], mh[1], mh[2], mh[3], store_policy);
            if (ERR) store_f4_first(e_lane + k * kSlotElems, e_out[0], e_out[1], e_out[2], e_out[3], store_policy);
        } else {
            if (FMT != FMT_INT4) *reinterpret_cast<uint32_t*>(w_lane + k * kSlotElems) = codes;
            else *reinterpret_cast<uint16_t*>(w_lane + k * (kSlotElems / 2)) = static_cast<uint16_t>(codes);
            *reinterpret_cast<float4*>(m_lane + k * kSlotElems) = make_float4(mh[0], mh[1], mh[2], mh[3]);
            if (ERR) *reinterpret_cast<float4*>(e_lane + k * kSlotElems) = make_float4(e_out[0], e_out[1], e_out[2], e_out[3]);
        }
    }
    return true;
}

// ---------------------------------------------------------------------------
// MODE_BLOCK        1x128 block scales, whole step in one pass
// MODE_BLOCK32      1x32 blocks (four per 128-element row) with power-of-two scales, whole step in one pass
// MODE_TENSOR_AMAX  per-tensor scale, pass 1: max |theta~| per tensor
// MODE_TENSOR_APPLY per-tensor scale, pass 2: quantize with the tensor's scale
// MODE_ROW          one scale per matrix row of up to 32 * 128 columns, whole step in one pass; a unit is
//                   floor(32 / R) whole matrix rows of R 128-element rows each
// Tensors handled here have a whole number of 128-element rows that start on
// 128-element boundaries (cols % 128 == 0, or a flat tensor with numel % 128 == 0).
// MODE_BLOCK32 takes power-of-two scales only; the other modes take f32 and bf16 scales only.
// ---------------------------------------------------------------------------
// ERR: the tensors carry error buffers (see eco_attach_error_buffers); a separate instantiation, so that the plain
// method pays nothing for the option.
template <int FMT, int OPT, int RND, int MODE, bool ERR>
// Adam: two CTAs per SM, so the compiler allows 96 registers per thread.  (112 would still add up to less than the
// register file, but the hardware was measured to place only one such CTA per SM.)  Momentum SGD carries no second
// moment and fits 72 registers without spilling: three CTAs per SM, i.e. 24 consumer warps to hide the latencies of
// its instruction-heavier bytes.
__global__ void __launch_bounds__(kStreamThreads, stream_ctas_per_sm<OPT, ERR>())
eco_stream_kernel(const TensorDesc* __restrict__ descs, const uint32_t* __restrict__ unit_tensor,
                  const uint32_t n_units, const StepParams P, const int scale_kind,
                  uint32_t* __restrict__ scratch_amax, uint32_t* __restrict__ scratch_amax_next,
                  float* __restrict__ scratch_s_old, const int reverse, const int interleave,
                  uint32_t* __restrict__ tickets, uint32_t* __restrict__ status) {
    using SL = StageLayout<FMT, OPT>;
    constexpr int S = SL::kStages;
    extern __shared__ __align__(128) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
    const uint32_t full0 = smem_addr(bars), empty0 = smem_addr(bars + S);
    uint8_t* stage0 = smem + SL::kBarriers;
    const uint32_t row_bars = smem_addr(smem + SL::kRowBars);
    float* xchg = reinterpret_cast<float*>(smem + SL::kExchange);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full0 + 8 * s, 2);                 // producer: expect_tx arrival + header/scales arrival
            mbar_init(empty0 + 8 * s, kConsumerWarps);
        }
        mbar_init(row_bars, kConsumerWarps);
        mbar_init(row_bars + 8, kConsumerWarps);
        mbar_init(smem_addr(smem + SL::kClusterBars), kConsumerWarps);       // one arrival per warp of this CTA, each announcing
        mbar_init(smem_addr(smem + SL::kClusterBars + 8), kConsumerWarps);   // the bytes the cluster sends for that warp
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const uint32_t csize = MODE == MODE_ROW ? cluster_size() : 1u, crank = MODE == MODE_ROW ? cluster_rank() : 0u;
    if (csize > 1) {
        // peers arrive on this CTA's barriers: nobody starts before every CTA of the cluster has initialised its own
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    }

    if (warp == kConsumerWarps) {
        // ------------------------------ producer ------------------------------
        // Units are handed out by a device-wide ticket counter, so CTAs that draw cheap units (tensors whose
        // gradient is all zero skip the square roots and divisions) simply draw more of them.  Ticket t maps to
        // unit (t mod W) * ceil(n / W) + t / W: W regions of the parameter set are walked at the same time, which
        // mixes compute-heavy and memory-heavy tensors on every SM.  tickets[0] counts tickets, tickets[1] CTAs
        // that are done drawing; the last one rewinds both for the next launch.
        const uint32_t W = static_cast<uint32_t>(interleave);
        const uint32_t per_region = div_ceil_u32(n_units, W);
        const uint32_t n_tickets = ticket_count(n_units, W);   // n_units < 2^31: fits, with room for the draws past the end
        auto draw = [&]() -> uint32_t {
            uint32_t t = 0;
            if (lane == 0) t = atomicAdd(tickets, 1u);
            return __shfl_sync(0xFFFFFFFFu, t, 0);
        };
        uint32_t it = 0;
        bool ok = true;
        // Stages one unit: waits for a free stage, issues the copies, writes the header.
        auto stage_unit = [&](const uint32_t unit) -> bool {
            const TensorDesc T = descs[__ldg(unit_tensor + unit)];
            const uint32_t s = it % S, ph = (it / S) & 1;
            if (!mbar_wait(empty0 + 8 * s, ph ^ 1, status, 1u)) return false;
            uint8_t* st = stage0 + static_cast<size_t>(s) * SL::kBytes;
            const uint32_t local = unit - T.first_unit;
            uint64_t row0, mrow0;
            uint32_t nrows, n_mrows, segs;
            if (MODE == MODE_ROW && csize > 1) {
                // the unit is ONE matrix row of R segments; this CTA takes segments [rank Rc, (rank + 1) Rc) of it
                const uint32_t R = T.blocks_per_row, Rc = div_ceil_u32(R, csize);
                const uint32_t lo = crank * Rc, hi = lo + Rc < R ? lo + Rc : R;
                row0 = static_cast<uint64_t>(local) * R + lo;
                nrows = hi - lo;
                mrow0 = local;
                n_mrows = 1u;
                segs = nrows;
            } else {
                const uint32_t unit_rows = MODE == MODE_ROW ? T.unit_rows : static_cast<uint32_t>(kUnitRows);
                row0 = static_cast<uint64_t>(local) * unit_rows;
                const uint64_t left = T.n_blocks - row0;
                nrows = left < unit_rows ? static_cast<uint32_t>(left) : unit_rows;
                const uint32_t mrows_per_unit = MODE == MODE_ROW ? unit_rows / T.blocks_per_row : 0u;
                mrow0 = static_cast<uint64_t>(local) * mrows_per_unit;
                n_mrows = MODE == MODE_ROW ? nrows / T.blocks_per_row : 0u;
                segs = T.blocks_per_row;
            }
            const uint32_t full = full0 + 8 * s;
            if (lane == 0) {
                const uint32_t cb = nrows * SL::kCodeRow, gb = nrows * 256u, mb = nrows * 512u;
                mbar_arrive_expect_tx(full, cb + gb + mb + (OPT == OPT_ADAM ? mb : 0u));
                bulk_load(smem_addr(st + SL::kCodes), T.w + row0 * SL::kCodeRow, cb, full);
                bulk_load(smem_addr(st + SL::kGrad), T.grad + row0 * 128, gb, full);
                bulk_load(smem_addr(st + SL::kM), T.m + row0 * 128, mb, full);
                if (OPT == OPT_ADAM) bulk_load(smem_addr(st + SL::kV), T.v + row0 * 128, mb, full);
                StageHeader h;
                h.w = T.w; h.scale = T.scale; h.m = T.m; h.v = T.v;
                h.row0 = row0; h.nrows = nrows; h.tensor_id = T.tensor_id; h.slot = T.slot;
                h.s_old = 1.0f; h.s_new = 1.0f; h.inv_new = 1.0f;
                h.seg_per_row = segs; h.div_magic = 65536u / segs + 1u;
                h.n_mrows = n_mrows; h.pass = 0u; h.barrier_target = 0u; h.first_of_tensor = 0u; h.mrow0 = mrow0; h.index_base = T.index_base; h.e = T.e;
                if (MODE == MODE_TENSOR_AMAX) {
                    h.s_old = load_scale(T.scale, 0, scale_kind);
                    if (local == 0) scratch_s_old[T.slot] = h.s_old;
                }
                if (MODE == MODE_TENSOR_APPLY) {
                    h.s_old = scratch_s_old[T.slot];
                    uint32_t bits;
                    make_scale_div<FMT>(__uint_as_float(scratch_amax[T.slot]), scale_kind == SCALE_KIND_BF16, h.s_new, h.inv_new, bits);
                    if (local == 0) {
                        store_scale(T.scale, 0, scale_kind, h.s_new, bits);
                        scratch_amax_next[T.slot] = 0u;
                    }
                }
                *reinterpret_cast<StageHeader*>(st + SL::kHeader) = h;
            }
            if (MODE == MODE_BLOCK && lane < static_cast<int>(nrows))
                reinterpret_cast<float*>(st + SL::kScales)[lane] = load_scale(T.scale, row0 + lane, scale_kind);
            if (MODE == MODE_BLOCK32) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (lane * 4 + j < static_cast<int>(nrows) * 4)
                        reinterpret_cast<float*>(st + SL::kScales)[lane * 4 + j] = load_scale(T.scale, row0 * 4 + lane * 4 + j, SCALE_KIND_E8M0);
            }
            if (MODE == MODE_ROW && lane < static_cast<int>(n_mrows))
                reinterpret_cast<float*>(st + SL::kScales)[lane] = load_scale(T.scale, mrow0 + lane, scale_kind);
            __syncwarp();
            if (lane == 0) mbar_arrive(full);
            ++it;
            return true;
        };
        if (MODE == MODE_ROW && csize > 1) {
            // a cluster works on one matrix row at a time, all its CTAs on the same one: cluster c of K takes the
            // rows c, c + K, ... of the launch (no tickets: the CTAs of a cluster must agree without talking)
            const uint32_t n_clusters = gridDim.x / csize, cid = blockIdx.x / csize;
            for (uint32_t unit = cid; unit < n_units && ok; unit += n_clusters) ok = stage_unit(unit);
        } else {
            uint32_t ticket = draw();
            while (ticket < n_tickets) {
                const uint32_t next_ticket = draw();          // in flight while this unit is set up
                const uint32_t cand = (ticket % W) * per_region + ticket / W;
                ticket = next_ticket;
                if (cand >= n_units) continue;
                ok = stage_unit(reverse ? (n_units - 1 - cand) : cand);
                if (!ok) break;
            }
            if (lane == 0 && atomicAdd(tickets + 1, 1u) == gridDim.x - 1) {
                tickets[0] = 0u;                               // every CTA has drawn its last ticket
                tickets[1] = 0u;
            }
        }
        if (ok) {
            // end marker: a stage whose header says "no rows"
            const uint32_t s = it % S, ph = (it / S) & 1;
            ok = mbar_wait(empty0 + 8 * s, ph ^ 1, status, 1u);
            if (ok && lane == 0) {
                uint8_t* st = stage0 + static_cast<size_t>(s) * SL::kBytes;
                reinterpret_cast<StageHeader*>(st + SL::kHeader)->nrows = 0u;
                mbar_arrive_expect_tx(full0 + 8 * s, 0u);
                mbar_arrive(full0 + 8 * s);
            }
        }
        if (!ok) {
            // leave only after the copies already issued have landed (bounded)
            const uint32_t pending = it < static_cast<uint32_t>(S) ? it : static_cast<uint32_t>(S);
            for (uint32_t k = 0; k < pending; ++k) {
                const uint32_t j = it - 1 - k;
                mbar_wait(full0 + 8 * (j % S), (j / S) & 1, status, 2u);
            }
        }
        return;
    }

    // -------------------------------- consumers --------------------------------
    uint32_t cur_slot = 0xFFFFFFFFu;
    float run_max = 0.0f;                         // MODE_TENSOR_AMAX
    for (uint32_t it = 0;; ++it) {
        const uint32_t s = it % S, ph = (it / S) & 1;
        if (!mbar_wait(full0 + 8 * s, ph, status, 3u)) return;
        const uint8_t* st = stage0 + static_cast<size_t>(s) * SL::kBytes;
        const StageHeader* h = reinterpret_cast<const StageHeader*>(st + SL::kHeader);
        const uint32_t empty = empty0 + 8 * s;
        const uint32_t nrows = h->nrows;
        if (nrows == 0u) break;                   // end marker
        bool ok;
        if constexpr (MODE == MODE_ROW) {
            // rows are dealt round-robin: this warp has rows warp, warp + 8, ... below nrows
            const int mine = static_cast<int>(nrows) > warp ? (static_cast<int>(nrows) - warp + kConsumerWarps - 1) / kConsumerWarps : 0;
            // (in a cluster: unit `it` uses exchange slot and barrier it & 1, whose phase parity is (it >> 1) & 1)
            // (the partial maxima of a cluster, 2 parities x 4 CTAs x 8 warps, lie where the single-CTA form keeps its
            // exchange arrays: a launch is one or the other)
            const ClusterInfo cl{crank, csize, smem_addr(smem + SL::kExchange), smem_addr(smem + SL::kClusterBars), (it >> 1) & 1u,
                                 reinterpret_cast<const float*>(smem + SL::kExchange)};
            const TensorScales none{1.0f, 1.0f, 1.0f};
            if (mine == 4)
                ok = consume_unit<FMT, OPT, RND, MODE, true, ERR, 4>(P, scale_kind, st, h, empty, warp, lane, scratch_amax, cur_slot,
                                                                     run_max, xchg, row_bars, it & 1u, status, none, 0, cl);
            else if (mine == 3)
                ok = consume_unit<FMT, OPT, RND, MODE, true, ERR, 3>(P, scale_kind, st, h, empty, warp, lane, scratch_amax, cur_slot,
                                                                     run_max, xchg, row_bars, it & 1u, status, none, 0, cl);
            else
                ok = consume_unit<FMT, OPT, RND, MODE, false, ERR, 4>(P, scale_kind, st, h, empty, warp, lane, scratch_amax, cur_slot,
                                                                      run_max, xchg, row_bars, it & 1u, status, none, 0, cl);
        } else if (nrows == kUnitRows)   // (discarded statement of the if constexpr above for the per-row mode)
            ok = consume_unit<FMT, OPT, RND, MODE, true, ERR>(P, scale_kind, st, h, empty, warp, lane, scratch_amax, cur_slot,
                                                              run_max, xchg, row_bars, it & 1u, status,
                                                              TensorScales{h->s_old, h->s_new, h->inv_new});
        else
            ok = consume_unit<FMT, OPT, RND, MODE, false, ERR>(P, scale_kind, st, h, empty, warp, lane, scratch_amax, cur_slot,
                                                               run_max, xchg, row_bars, it & 1u, status,
                                                               TensorScales{h->s_old, h->s_new, h->inv_new});
        if (!ok) return;
    }
    if (MODE == MODE_TENSOR_AMAX && cur_slot != 0xFFFFFFFFu) {
        const float z = warp_amax(run_max);
        if (lane == 0) atomicMax(scratch_amax + cur_slot, __float_as_uint(z));
    }
}

// ---------------------------------------------------------------------------
// Per-tensor scale in ONE cooperative launch: the parameter set is cut into waves of whole tensors whose inputs
// are about as large as L2 (a tensor larger than that is a wave of its own).  Wave by wave, every CTA streams its
// share of the wave's units once for max |theta~| (pass 1), the grid meets at a barrier, and the CTA goes over the
// same units again (pass 2) with the now complete maxima: first the units still sitting in its shared-memory stages
// (no load at all), then the others newest first, which the L2 still holds for the most part.  A tensor that fits
// the chip is therefore read from HBM once (20 B/param for FP8 + Adam) instead of twice (31).
//
// CTA c of G owns units c, c + G, ... of every wave: the same SM touches the same addresses in both passes.
// The producer warp publishes a sequence of stages (round-robin over the ring); a publication is one of
//   WAVE_AMAX    a freshly loaded unit, pass 1
//   WAVE_APPLY   a unit for pass 2: freshly loaded, or -- `resident` -- the stage as pass 1 left it (nothing is copied)
//   WAVE_NOOP    nothing (keeps the ring position in step when a CTA has fewer units in a wave than stages)
//   WAVE_END     end of the kernel
// The first pass-2 publication of a wave (a no-op if the CTA has no unit there) carries the barrier: before they
// process it, the consumer warps post their maxima, one thread arrives on the grid counter and waits, bounded, until
// every CTA has arrived.  The producer never waits for the grid: it goes on issuing the copies of pass 2 while the
// consumers stand at the barrier, so the memory system stays busy across it.  Launched cooperatively, so that all
// CTAs are resident and the barrier can complete.
// L2 hints (measured with a probe of this access pattern): the units that will stay in shared memory, the re-loads of
// pass 2 and all stores are marked evict-first, which leaves the L2 to the lines pass 2 still needs.
// ---------------------------------------------------------------------------
enum : uint32_t { WAVE_AMAX = 1, WAVE_APPLY = 2, WAVE_NOOP = 3, WAVE_END = 4 };

#ifdef ECO_WAVE_TRACE
// Development aid, not compiled into the library: nanosecond timestamps of every CTA at four points of every wave
// (first unit of pass 1 in hand, arrival at the barrier, release from it, first unit of the next wave in hand).
constexpr uint32_t kTraceWaves = 128, kTraceCtas = 512;
__device__ unsigned long long g_wave_trace[kTraceCtas * kTraceWaves * 4];
__device__ __forceinline__ void wave_trace(uint32_t wave, int point) {
    if (threadIdx.x == 0 && wave < kTraceWaves && blockIdx.x < kTraceCtas) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
        g_wave_trace[(blockIdx.x * kTraceWaves + wave) * 4 + point] = t;
    }
}
#define ECO_TRACE(wave, point) wave_trace(wave, point)
#else
#define ECO_TRACE(wave, point)
#endif
constexpr uint32_t kGridBarrierTimeout = 6u;       // status code

// Meeting point of the 8 consumer warps of a CTA on an mbarrier of its own (count 8), bounded like every other wait.
__device__ __forceinline__ bool consumers_sync(uint32_t bar, uint32_t& phase, int lane, uint32_t* status) {
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
    const bool ok = mbar_wait(bar, phase & 1u, status, 8u);
    ++phase;
    return ok;
}

// Bounded grid barrier for the consumer warps of a CTA: they meet, one thread arrives on the grid counter and waits
// until every CTA has, they meet again.  Returns false when a wait ran out (the code is in *status).
__device__ __forceinline__ bool wave_grid_barrier(uint32_t* counter, uint32_t target, uint32_t* status, uint32_t* abort_flag,
                                                  uint32_t bar, uint32_t& phase, int lane,
                                                  long long limit_cycles = kWaitLimitCycles) {
    if (!consumers_sync(bar, phase, lane, status)) return false;         // every warp has posted its maxima
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1u);
        const long long t0 = clock64();
        uint32_t seen;
        for (;;) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
            if (seen >= target) break;
            if (clock64() - t0 > limit_cycles) {
                atomicExch(status, kGridBarrierTimeout);
                *reinterpret_cast<volatile uint32_t*>(abort_flag) = 1u;
                break;
            }
        }
        __threadfence();
    }
    if (!consumers_sync(bar, phase, lane, status)) return false;
    return *reinterpret_cast<volatile uint32_t*>(abort_flag) == 0u;
}

template <int FMT, int OPT, int RND, bool ERR>
__global__ void __launch_bounds__(kStreamThreads, stream_ctas_per_sm<OPT, ERR>())
eco_wave_kernel(const TensorDesc* __restrict__ descs, const uint32_t* __restrict__ unit_tensor,
                const WaveDesc* __restrict__ waves, const uint32_t n_waves, const StepParams P, const int scale_kind,
                uint32_t* __restrict__ scratch_amax, uint32_t* __restrict__ scratch_amax_next,
                float* __restrict__ scratch_s_old, uint32_t* __restrict__ grid_counter, uint32_t* __restrict__ wave_tickets,
                uint32_t* __restrict__ status) {
    using SL = StageLayout<FMT, OPT>;
    constexpr int S = SL::kStages;
    extern __shared__ __align__(128) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
    const uint32_t full0 = smem_addr(bars), empty0 = smem_addr(bars + S);
    uint8_t* stage0 = smem + SL::kBarriers;
    uint32_t* abort_flag = reinterpret_cast<uint32_t*>(smem + SL::kExchange);
    const bool dynamic = wave_tickets != nullptr;
    const uint32_t sync_bar = smem_addr(smem + SL::kRowBars);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t G = gridDim.x, cta = blockIdx.x;
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full0 + 8 * s, 2);
            mbar_init(empty0 + 8 * s, kConsumerWarps);
        }
        mbar_init(sync_bar, kConsumerWarps);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == kConsumerWarps) {
        // ------------------------------ producer ------------------------------
        const uint64_t evict_first = policy_evict_first();
        uint32_t it = 0;                         // publications so far; the next one goes to stage it % S
        uint32_t stage_unit[S];                  // unit (index inside the wave's share) a stage holds from pass 1, or none
        bool ok = true;
        // Publishes one stage.  load: copy the unit's inputs in; otherwise the stage keeps what it holds.
        uint32_t cur_ti = 0xFFFFFFFFu;           // tensor whose descriptor is in T
        TensorDesc T;
        float cur_s_old = 1.0f;
        auto publish = [&](uint32_t pass, uint32_t unit, bool load, bool hint, uint32_t barrier_target) -> bool {
            const uint32_t s = it % S, ph = (it / S) & 1;
            if (load) {
                // the descriptor is fetched BEFORE the wait for the stage, so that its latency hides behind that wait
                const uint32_t ti = __ldg(unit_tensor + unit);
                if (ti != cur_ti) {
                    T = descs[ti];
                    cur_ti = ti;
                    // (read in pass 1, where the tensor's old scale is still in place; a descriptor first met in pass 2
                    // reads the new one, which nothing uses)
                    cur_s_old = load_scale(T.scale, 0, scale_kind);
                }
            }
            if (!mbar_wait(empty0 + 8 * s, ph ^ 1, status, 1u)) return false;
            uint8_t* st = stage0 + static_cast<size_t>(s) * SL::kBytes;
            const uint32_t full = full0 + 8 * s;
            if (pass == WAVE_NOOP || pass == WAVE_END) {
                if (lane == 0) {
                    StageHeader* h = reinterpret_cast<StageHeader*>(st + SL::kHeader);
                    h->pass = pass;
                    h->barrier_target = barrier_target;
                    h->nrows = 0u;
                    mbar_arrive_expect_tx(full, 0u);
                }
            } else if (!load) {
                if (lane == 0) {                 // the stage as pass 1 left it: only the header changes
                    StageHeader* h = reinterpret_cast<StageHeader*>(st + SL::kHeader);
                    h->pass = pass;
                    h->barrier_target = barrier_target;
                    mbar_arrive_expect_tx(full, 0u);
                }
            } else {
                const uint32_t local = unit - T.first_unit;
                const uint64_t row0 = static_cast<uint64_t>(local) * kUnitRows;
                const uint64_t left = T.n_blocks - row0;
                const uint32_t nrows = left < kUnitRows ? static_cast<uint32_t>(left) : static_cast<uint32_t>(kUnitRows);
                if (lane == 0) {
                    const uint32_t cb = nrows * SL::kCodeRow, gb = nrows * 256u, mb = nrows * 512u;
                    mbar_arrive_expect_tx(full, cb + gb + mb + (OPT == OPT_ADAM ? mb : 0u));
                    if (hint) {
                        bulk_load_hint(smem_addr(st + SL::kCodes), T.w + row0 * SL::kCodeRow, cb, full, evict_first);
                        bulk_load_hint(smem_addr(st + SL::kGrad), T.grad + row0 * 128, gb, full, evict_first);
                        bulk_load_hint(smem_addr(st + SL::kM), T.m + row0 * 128, mb, full, evict_first);
                        if (OPT == OPT_ADAM) bulk_load_hint(smem_addr(st + SL::kV), T.v + row0 * 128, mb, full, evict_first);
                    } else {
                        bulk_load(smem_addr(st + SL::kCodes), T.w + row0 * SL::kCodeRow, cb, full);
                        bulk_load(smem_addr(st + SL::kGrad), T.grad + row0 * 128, gb, full);
                        bulk_load(smem_addr(st + SL::kM), T.m + row0 * 128, mb, full);
                        if (OPT == OPT_ADAM) bulk_load(smem_addr(st + SL::kV), T.v + row0 * 128, mb, full);
                    }
                    StageHeader h;
                    h.w = T.w; h.scale = T.scale; h.m = T.m; h.v = T.v;
                    h.row0 = row0; h.nrows = nrows; h.tensor_id = T.tensor_id; h.slot = T.slot;
                    h.s_old = 1.0f; h.s_new = 1.0f; h.inv_new = 1.0f;
                    h.seg_per_row = 1u; h.div_magic = 0u; h.n_mrows = 0u; h.pass = pass; h.mrow0 = 0u;
                    h.index_base = T.index_base; h.e = T.e;
                    h.barrier_target = barrier_target; h.first_of_tensor = local == 0u ? 1u : 0u;
                    if (pass == WAVE_AMAX) {
                        // the old scale: nobody stores this tensor's new one before the wave's barrier
                        h.s_old = cur_s_old;
                        if (local == 0) scratch_s_old[T.slot] = cur_s_old;
                    }
                    *reinterpret_cast<StageHeader*>(st + SL::kHeader) = h;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(full);
            ++it;
            return true;
        };
        // Several waves: the units of each pass of a wave are handed out by a ticket counter (two per wave), so that
        // every CTA is busy until the pass runs dry and all reach the barrier together; pass 2 walks the wave newest
        // first and finds it in L2.  (With the static split below, CTAs that are a little slower -- or hold one unit
        // more -- keep the whole grid waiting at every barrier.)
        auto draw = [&](uint32_t* counter) -> uint32_t {
            uint32_t t = 0;
            if (lane == 0) t = atomicAdd(counter, 1u);
            return __shfl_sync(0xFFFFFFFFu, t, 0);
        };
        for (uint32_t w = 0; dynamic && w < n_waves && ok; ++w) {
            const uint32_t first = waves[w].first_unit, n = waves[w].n_units;
            uint32_t t = draw(wave_tickets + 2 * w);
            while (t < n && ok) {
                const uint32_t tn = draw(wave_tickets + 2 * w);           // in flight while this unit is staged
                ok = publish(WAVE_AMAX, first + t, true, false, 0u);
                t = tn;
            }
            if (!ok) break;
            const uint32_t target = (w + 1u) * G;
            t = draw(wave_tickets + 2 * w + 1);
            if (t >= n) ok = publish(WAVE_NOOP, 0u, false, false, target);   // nothing left for this CTA: only the barrier
            bool first_pub = true;
            while (t < n && ok) {
                const uint32_t tn = draw(wave_tickets + 2 * w + 1);
                ok = publish(WAVE_APPLY, first + (n - 1u - t), true, true, first_pub ? target : 0u);
                first_pub = false;
                t = tn;
            }
        }
        // A single wave: static split, so that what a CTA streamed in pass 1 is still in its stages for pass 2.
        for (uint32_t w = 0; !dynamic && w < n_waves && ok; ++w) {
            const uint32_t first = waves[w].first_unit, n = waves[w].n_units;
            const uint32_t mine = n > cta ? (n - cta + G - 1) / G : 0u;          // units first + cta + j G, j < mine
#pragma unroll
            for (int s = 0; s < S; ++s) stage_unit[s] = 0xFFFFFFFFu;
            // pass 1; the units that end it in the stages are not needed from L2 again
            for (uint32_t j = 0; j < mine && ok; ++j) {
                stage_unit[it % S] = j;
                ok = publish(WAVE_AMAX, first + cta + j * G, true, j + S >= mine, 0u);
            }
            if (!ok) break;
            // pass 2: one round over the ring for what it still holds (at least one publication: it carries the barrier)
            const uint32_t target = (w + 1u) * G;
            uint32_t resident = mine < static_cast<uint32_t>(S) ? mine : static_cast<uint32_t>(S), k = 0;
            do {
                const uint32_t u = stage_unit[it % S];
                const uint32_t bt = k == 0 ? target : 0u;
                if (u != 0xFFFFFFFFu) {
                    stage_unit[it % S] = 0xFFFFFFFFu;
                    --resident;
                    ok = publish(WAVE_APPLY, first + cta + u * G, false, false, bt);
                } else {
                    ok = publish(WAVE_NOOP, 0u, false, false, bt);
                }
                ++k;
            } while (resident > 0 && ok);
            // the rest of pass 2, newest first
            if (mine > static_cast<uint32_t>(S))
                for (uint32_t j = mine - S; j-- > 0 && ok;)
                    ok = publish(WAVE_APPLY, first + cta + j * G, true, true, 0u);
        }
        if (ok) ok = publish(WAVE_END, 0u, false, false, 0u);
        if (!ok) {
            const uint32_t pending = it < static_cast<uint32_t>(S) ? it : static_cast<uint32_t>(S);
            for (uint32_t k = 0; k < pending; ++k) {
                const uint32_t j = it - 1 - k;
                mbar_wait(full0 + 8 * (j % S), (j / S) & 1, status, 2u);
            }
        }
        return;
    }

    // -------------------------------- consumers --------------------------------
    const uint64_t evict_first = policy_evict_first();
    uint32_t cur_slot = 0xFFFFFFFFu;
    float run_max = 0.0f;
    uint32_t sync_phase = 0u;
#ifdef ECO_WAVE_TRACE
    uint32_t trace_wave = 0u;
    bool trace_open = false;
#endif
    uint32_t scale_slot = 0xFFFFFFFFu;            // tensor whose scales are in ts
    TensorScales ts{1.0f, 1.0f, 1.0f};
    for (uint32_t it = 0;; ++it) {
        const uint32_t s = it % S, ph = (it / S) & 1;
        if (!mbar_wait(full0 + 8 * s, ph, status, 3u)) return;
        const uint8_t* st = stage0 + static_cast<size_t>(s) * SL::kBytes;
        const StageHeader* h = reinterpret_cast<const StageHeader*>(st + SL::kHeader);
        const uint32_t empty = empty0 + 8 * s;
        const uint32_t pass = h->pass, nrows = h->nrows, target = h->barrier_target;
        if (pass == WAVE_END) break;
#ifdef ECO_WAVE_TRACE
        if (pass == WAVE_AMAX && !trace_open) { ECO_TRACE(trace_wave, 0); trace_open = true; }
        if (target != 0u) ECO_TRACE(trace_wave, 1);
#endif
        if (target != 0u) {
            // end of this CTA's pass 1 of the wave: post the running maximum, then meet the other CTAs
            if (cur_slot != 0xFFFFFFFFu) {
                const float z = warp_amax(run_max);
                if (lane == 0) atomicMax(scratch_amax + cur_slot, __float_as_uint(z));
                cur_slot = 0xFFFFFFFFu;
                run_max = 0.0f;
            }
            scale_slot = 0xFFFFFFFFu;
            if (!wave_grid_barrier(grid_counter, target, status, abort_flag, sync_bar, sync_phase, lane)) return;
#ifdef ECO_WAVE_TRACE
            ECO_TRACE(trace_wave, 2);
            ++trace_wave;
            trace_open = false;
#endif
        }
        if (pass == WAVE_NOOP) {
            __syncwarp();
            if (lane == 0) mbar_arrive(empty);
            continue;
        }
        bool ok;
        if (pass == WAVE_AMAX) {
            const TensorScales t1{h->s_old, 1.0f, 1.0f};
            if (nrows == kUnitRows)
                ok = consume_unit<FMT, OPT, RND, MODE_TENSOR_AMAX, true, false>(P, scale_kind, st, h, empty, warp, lane, scratch_amax,
                                                                                cur_slot, run_max, nullptr, 0u, 0u, status, t1);
            else
                ok = consume_unit<FMT, OPT, RND, MODE_TENSOR_AMAX, false, false>(P, scale_kind, st, h, empty, warp, lane, scratch_amax,
                                                                                 cur_slot, run_max, nullptr, 0u, 0u, status, t1);
        } else {
            const uint32_t slot = h->slot;
            if (slot != scale_slot) {
                // the tensor's maximum is complete (barrier passed); its old scale was saved in pass 1 by the owner
                // of its first unit.  Both were written by other SMs: read past the L1.
                scale_slot = slot;
                uint32_t bits;
                ts.s_old = __ldcg(scratch_s_old + slot);
                make_scale_div<FMT>(__uint_as_float(__ldcg(scratch_amax + slot)), scale_kind == SCALE_KIND_BF16, ts.s_new, ts.inv_new, bits);
                if (h->first_of_tensor && warp == 0 && lane == 0) {
                    store_scale(h->scale, 0, scale_kind, ts.s_new, bits);
                    scratch_amax_next[slot] = 0u;
                }
            } else if (h->first_of_tensor && warp == 0 && lane == 0) {
                uint32_t bits;
                float s_new, inv_new;
                make_scale_div<FMT>(__uint_as_float(__ldcg(scratch_amax + slot)), scale_kind == SCALE_KIND_BF16, s_new, inv_new, bits);
                store_scale(h->scale, 0, scale_kind, s_new, bits);
                scratch_amax_next[slot] = 0u;
            }
            if (nrows == kUnitRows)
                ok = consume_unit<FMT, OPT, RND, MODE_TENSOR_APPLY, true, ERR, 4, true>(P, scale_kind, st, h, empty, warp, lane, scratch_amax,
                                                                                       cur_slot, run_max, nullptr, 0u, 0u, status, ts, evict_first);
            else
                ok = consume_unit<FMT, OPT, RND, MODE_TENSOR_APPLY, false, ERR, 4, true>(P, scale_kind, st, h, empty, warp, lane, scratch_amax,
                                                                                        cur_slot, run_max, nullptr, 0u, 0u, status, ts, evict_first);
        }
        if (!ok) return;
    }
    // the last CTA out rewinds the grid counter for the next launch (every CTA has passed every barrier by then)
    if (!consumers_sync(sync_bar, sync_phase, lane, status)) return;
    if (threadIdx.x == 0 && atomicAdd(grid_counter + 1, 1u) == G - 1) {
        grid_counter[0] = 0u;
        grid_counter[1] = 0u;
        if (dynamic)
            for (uint32_t k = 0; k < 2u * n_waves; ++k) wave_tickets[k] = 0u;
    }
}

template <int FMT, int OPT, int RND, bool ERR>
static cudaError_t launch_wave_one(const TensorDesc* descs, const uint32_t* unit_tensor, const WaveDesc* waves, uint32_t n_waves,
                                   const StepParams& P, int scale_kind, uint32_t* amax, uint32_t* amax_next, float* s_old,
                                   uint32_t* grid_counter, uint32_t* wave_tickets, uint32_t* status, int grid_cap, int sm_count,
                                   cudaStream_t stream) {
    using SL = StageLayout<FMT, OPT>;
    static int resident = -1;                     // CTAs of this instantiation that fit one SM
    auto kernel = eco_wave_kernel<FMT, OPT, RND, ERR>;
    if (resident < 0) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::kSmem);
        if (e != cudaSuccess) return e;
        int n = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, kStreamThreads, SL::kSmem);
        if (e != cudaSuccess) return e;
        if (n < 1) return cudaErrorLaunchOutOfResources;
        resident = n < stream_ctas_per_sm<OPT, ERR>() ? n : stream_ctas_per_sm<OPT, ERR>();
    }
    // every CTA must be resident for the grid barrier: never more than the SMs can hold at once
    int grid = resident * sm_count;
    if (grid_cap > 0 && grid_cap < grid) grid = grid_cap;
    StepParams Pc = P;
    int sk = scale_kind;
    void* args[] = {&descs, &unit_tensor, &waves, &n_waves, &Pc, &sk, &amax, &amax_next, &s_old, &grid_counter, &wave_tickets, &status};
    return cudaLaunchCooperativeKernel(reinterpret_cast<void*>(kernel), dim3(grid), dim3(kStreamThreads), args, SL::kSmem, stream);
}

// ---------------------------------------------------------------------------
template <int FMT, int OPT, int RND, int MODE, bool ERR = false>
static cudaError_t launch_one(const TensorDesc* descs, const uint32_t* unit_tensor, uint32_t n_units, const StepParams& P,
                              int scale_kind, uint32_t* amax, uint32_t* amax_next, float* s_old, bool reverse,
                              uint32_t* tickets, uint32_t* status, int grid_cap, int sm_count, cudaStream_t stream,
                              int cluster = 1) {
    using SL = StageLayout<FMT, OPT>;
    static bool configured = false;
    auto kernel = eco_stream_kernel<FMT, OPT, RND, MODE, ERR>;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::kSmem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const uint32_t cap = static_cast<uint32_t>(grid_cap > 0 ? grid_cap : sm_count * stream_ctas_per_sm<OPT, ERR>());
    const int interleave = (MODE == MODE_BLOCK || MODE == MODE_BLOCK32 || MODE == MODE_ROW) ? kInterleave : 1;
    if (cluster > 1) {
        // per-row scales on rows of several units: clusters of `cluster` CTAs, one matrix row per cluster at a time
        const uint32_t c = static_cast<uint32_t>(cluster);
        uint32_t n_clusters = cap / c;
        if (n_clusters > n_units) n_clusters = n_units;
        if (n_clusters == 0) return cudaErrorInvalidConfiguration;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(n_clusters * c);
        cfg.blockDim = dim3(kStreamThreads);
        cfg.dynamicSmemBytes = SL::kSmem;
        cfg.stream = stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = c;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, kernel, descs, unit_tensor, n_units, P, scale_kind, amax, amax_next, s_old,
                                  reverse ? 1 : 0, interleave, tickets, status);
    }
    const uint32_t grid = n_units < cap ? n_units : cap;
    kernel<<<grid, kStreamThreads, SL::kSmem, stream>>>(descs, unit_tensor, n_units, P, scale_kind, amax, amax_next,
                                                        s_old, reverse ? 1 : 0, interleave, tickets, status);
    return cudaGetLastError();
}

#define ECO_S_FMT(fmt, ...)                                            \
    if ((fmt) == FMT_FP8) { constexpr int F = FMT_FP8; __VA_ARGS__ }   \
    else if ((fmt) == FMT_E5M2) { constexpr int F = FMT_E5M2; __VA_ARGS__ } \
    else { constexpr int F = FMT_INT4; __VA_ARGS__ }
#define ECO_S_OPT(opt, ...)                                              \
    if ((opt) == OPT_SGDM) { constexpr int O = OPT_SGDM; __VA_ARGS__ }   \
    else { constexpr int O = OPT_ADAM; __VA_ARGS__ }
#define ECO_S_RND(rnd, ...)                                            \
    if ((rnd) == RND_RTN) { constexpr int R = RND_RTN; __VA_ARGS__ }   \
    else { constexpr int R = RND_SR; __VA_ARGS__ }

cudaError_t launch_stream(const LaunchConfig& c, int mode, const TensorDesc* descs, const uint32_t* unit_tensor,
                          uint32_t n_units, const StepParams& P, uint32_t* amax, uint32_t* amax_next, float* s_old,
                          bool reverse, uint32_t* tickets, uint32_t* status, int grid_cap, cudaStream_t stream,
                          bool with_errors, int cluster) {
    if (n_units == 0) return cudaSuccess;
    if (mode == STREAM_TENSOR_AMAX) {
        ECO_S_FMT(c.format, ECO_S_OPT(c.optimizer, {
            return launch_one<F, O, RND_RTN, MODE_TENSOR_AMAX>(descs, unit_tensor, n_units, P, c.scale_kind, amax,
                                                               amax_next, s_old, reverse, tickets, status, grid_cap, c.sm_count, stream);
        }))
    }
#define ECO_S_LAUNCH(MODE_, ERR_)                                                                                      \
    return launch_one<F, O, R, MODE_, ERR_>(descs, unit_tensor, n_units, P, c.scale_kind, amax, amax_next, s_old, reverse, \
                                            tickets, status, grid_cap, c.sm_count, stream, MODE_ == MODE_ROW ? cluster : 1)
    ECO_S_FMT(c.format, ECO_S_OPT(c.optimizer, ECO_S_RND(c.rounding, {
        if (with_errors) {
            if (mode == STREAM_ROW) ECO_S_LAUNCH(MODE_ROW, true);
            if (mode == STREAM_BLOCK) ECO_S_LAUNCH(MODE_BLOCK, true);
            if (mode == STREAM_BLOCK32) ECO_S_LAUNCH(MODE_BLOCK32, true);
            ECO_S_LAUNCH(MODE_TENSOR_APPLY, true);
        }
        if (mode == STREAM_ROW) ECO_S_LAUNCH(MODE_ROW, false);
        if (mode == STREAM_BLOCK) ECO_S_LAUNCH(MODE_BLOCK, false);
        if (mode == STREAM_BLOCK32) ECO_S_LAUNCH(MODE_BLOCK32, false);
        ECO_S_LAUNCH(MODE_TENSOR_APPLY, false);
    })))
#undef ECO_S_LAUNCH
    return cudaErrorInvalidValue;
}

#ifdef ECO_WAVE_TRACE
extern "C" int eco_debug_read_wave_trace(void* host, size_t bytes) {
    return static_cast<int>(cudaMemcpyFromSymbol(host, g_wave_trace, bytes < sizeof(g_wave_trace) ? bytes : sizeof(g_wave_trace)));
}
#endif

cudaError_t launch_wave(const LaunchConfig& c, const TensorDesc* descs, const uint32_t* unit_tensor, const WaveDesc* waves,
                        uint32_t n_waves, const StepParams& P, uint32_t* amax, uint32_t* amax_next, float* s_old,
                        uint32_t* grid_counter, uint32_t* wave_tickets, uint32_t* status, int grid_cap, cudaStream_t stream,
                        bool with_errors) {
    if (n_waves == 0) return cudaSuccess;
    ECO_S_FMT(c.format, ECO_S_OPT(c.optimizer, ECO_S_RND(c.rounding, {
        if (with_errors)
            return launch_wave_one<F, O, R, true>(descs, unit_tensor, waves, n_waves, P, c.scale_kind, amax, amax_next, s_old,
                                                  grid_counter, wave_tickets, status, grid_cap, c.sm_count, stream);
        return launch_wave_one<F, O, R, false>(descs, unit_tensor, waves, n_waves, P, c.scale_kind, amax, amax_next, s_old,
                                               grid_counter, wave_tickets, status, grid_cap, c.sm_count, stream);
    })))
    return cudaErrorInvalidValue;
}

// Self-test of the bounded wait: one warp waits on an mbarrier that nothing ever arrives on.  The wait
// must give up after limit_cycles, record its code and let the kernel end normally.
__global__ void eco_wait_selftest_kernel(uint32_t* status, long long limit_cycles) {
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_addr(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    mbar_wait(smem_addr(&bar), 0, status, 7u, limit_cycles);
}

// Self-test of the bounded grid barrier: two CTAs of 8 warps meet at a barrier that expects three arrivals.  The
// wait must give up after limit_cycles, record code 6 and let the kernel end normally.
__global__ void __launch_bounds__(kConsumerWarps * 32) eco_grid_wait_selftest_kernel(uint32_t* counter, uint32_t* status, long long limit_cycles) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_addr(&bar), kConsumerWarps);
        abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    uint32_t phase = 0u;
    wave_grid_barrier(counter, gridDim.x + 1u, status, &abort_flag, smem_addr(&bar), phase, threadIdx.x & 31, limit_cycles);
}

cudaError_t launch_grid_wait_selftest(uint32_t* counter, uint32_t* status, long long limit_cycles, cudaStream_t stream) {
    eco_grid_wait_selftest_kernel<<<2, kConsumerWarps * 32, 0, stream>>>(counter, status, limit_cycles);
    return cudaGetLastError();
}

cudaError_t launch_wait_selftest(uint32_t* status, long long limit_cycles, cudaStream_t stream) {
    eco_wait_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_cycles);
    return cudaGetLastError();
}

int stream_unit_rows() { return kUnitRows; }
int stream_max_cluster() { return 4; }

}  // namespace eco
