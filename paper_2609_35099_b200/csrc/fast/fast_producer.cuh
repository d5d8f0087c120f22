// The producer side of the specialised kernels (forward and backward share it).
//
// A tile of the ring is "full" when the arrival that announces its bulk copies, their bytes, and the arrival
// after the tile's tables (receiver ids, change mask, A entries) are in.  The
// work is two parts, CopyPart and TablePart, run either by two warps (copy_producer + table_producer:
// the copies of a freed slot are issued without waiting for table work) or by one warp
// (combined_producer: less hot code, one warp fewer).
//
// L describes the shared-memory ring (T, NS, S_EDGE, X_EDGE, off_bar, off_abort, off_stage, stage_bytes and the
// offsets st_s / st_x / st_A / st_y / st_r inside a stage; with L::DBL also st_us / st_ux / st_B / st_uy for the
// cotangents that the fused double backward stages beside the primal inputs); Tab gives the A-slot tables of the kernel
// (APAD, DSH, pair_rec, rec_val, rec_i2); P is the kernel's parameter struct (x, sh, w, senders, receivers,
// identity, status).
#pragma once
#include "harmonics.cuh"
#include "fast_common.cuh"

namespace e3j {
namespace fast {

// Per A slot: up to two records, A = c0 * y[i2_0] + c1 * y[i2_1].
struct ASlot {
    float c0, c1;
    int i2_0, i2_1;
};

// ------------------------------------------------------------------------ copies of one tile
template <class L, class P>
struct CopyPart {
    static constexpr int T = L::T;
    const P& p;
    const int lane;
    const int64_t e_begin, e_end;
    const int n_tiles;
    int snd_a = 0, snd_b = 0;   // sender ids of the next two tiles (lane i: edge i of the tile)

    __device__ __forceinline__ CopyPart(const P& p_, int lane_, int64_t b, int64_t e, int n)
        : p(p_), lane(lane_), e_begin(b), e_end(e), n_tiles(n) {
        load(0, snd_a);
        load(1, snd_b);
    }
    __device__ __forceinline__ void load(int t, int& snd) {
        if (t >= n_tiles) return;
        const int64_t e0 = e_begin + (int64_t)t * T;
        const int n_e = (int)min((int64_t)T, e_end - e0);
        if (lane < n_e) snd = p.identity ? (int)(e0 + lane) : p.senders[e0 + lane];
    }
    // The tile's weights are one bulk copy, every gathered sender row another (issued by its own lane);
    // the barrier counts their bytes.  (16-byte asynchronous copies for the rows were measured slower in the
    // backward: they share the load/store pipe with the consumers.)
    __device__ __forceinline__ void issue(int t, unsigned char* st, uint64_t* full_bar) {
        const int64_t e0 = e_begin + (int64_t)t * T;
        const int n_e = (int)min((int64_t)T, e_end - e0);
        if (lane == 0) {
            // arrival and byte count in one step: the phase cannot complete before the bytes are expected
            mbar_arrive_expect_tx(full_bar, (uint32_t)n_e * 4u * (L::DBL ? 2u : 1u) * (L::S_EDGE + L::X_EDGE));
            bulk_g2s(st + L::st_s, p.w + (size_t)e0 * L::S_EDGE, (uint32_t)n_e * 4u * L::S_EDGE, full_bar);
        }
        if (lane < n_e)
            bulk_g2s(st + L::st_x + (size_t)lane * 4 * L::X_EDGE, p.x + (size_t)snd_a * L::X_EDGE, 4u * L::X_EDGE,
                     full_bar);
        if constexpr (L::DBL) {
            if (lane == 31)
                bulk_g2s(st + L::st_us, p.ct_w + (size_t)e0 * L::S_EDGE, (uint32_t)n_e * 4u * L::S_EDGE, full_bar);
            if (lane < n_e)
                bulk_g2s(st + L::st_ux + (size_t)lane * 4 * L::X_EDGE, p.ct_x + (size_t)snd_a * L::X_EDGE,
                         4u * L::X_EDGE, full_bar);
        }
        snd_a = snd_b;
        load(t + 2, snd_b);   // two tiles ahead of its use
    }
};

// ------------------------------------------------------------------------ tables of one tile
template <class L, class Tab, class P>
struct TablePart {
    static constexpr int T = L::T;
    static constexpr int YPL = (T * Tab::DSH + 31) / 32;
    static constexpr int NA = (Tab::APAD + 31) / 32;
    const P& p;
    const int lane;
    const int64_t e_begin, e_end;
    const int n_tiles;
    ASlot tab[NA];              // this lane's A slots (lane, lane + 32, ...)
    int rcv_a = -1, rcv_b = -1; // receiver ids of the next two tiles
    float y_a[YPL], y_b[YPL];   // harmonics of the next two tiles
    float v_a[3], v_b[3];       // or, when the call gives edge vectors instead, lane j's vector of each tile
    float uy_a[L::DBL ? YPL : 1], uy_b[L::DBL ? YPL : 1];   // and their cotangents (double backward)
    int last_rcv = -1;

    __device__ __forceinline__ TablePart(const P& p_, int lane_, int64_t b, int64_t e, int n)
        : p(p_), lane(lane_), e_begin(b), e_end(e), n_tiles(n) {
#pragma unroll
        for (int i = 0; i < NA; ++i) {
            const int slot = lane + 32 * i;
            ASlot a{0.f, 0.f, 0, 0};
            if (slot < Tab::APAD) {
                const PairRec pr = Tab::pair_rec(slot);
                if (pr.count > 0) { a.c0 = Tab::rec_val(pr.start); a.i2_0 = Tab::rec_i2(pr.start); }
                if (pr.count > 1) { a.c1 = Tab::rec_val(pr.start + 1); a.i2_1 = Tab::rec_i2(pr.start + 1); }
            }
            tab[i] = a;
        }
        load(0, rcv_a, y_a, v_a);
        load(1, rcv_b, y_b, v_b);
        if constexpr (L::DBL) { load_ct(0, uy_a); load_ct(1, uy_b); }
    }
    __device__ __forceinline__ void load_ct(int t, float (&yv)[L::DBL ? YPL : 1]) {
        if (t >= n_tiles) return;
        const int64_t e0 = e_begin + (int64_t)t * T;
        const int n_e = (int)min((int64_t)T, e_end - e0);
#pragma unroll
        for (int i = 0; i < (L::DBL ? YPL : 0); ++i) {
            const int idx = i * 32 + lane;
            if (idx < n_e * Tab::DSH) yv[i] = p.ct_sh[e0 * Tab::DSH + idx];
        }
    }
    __device__ __forceinline__ void load(int t, int& rcv, float (&yv)[YPL], float (&vv)[3]) {
        if (t >= n_tiles) return;
        const int64_t e0 = e_begin + (int64_t)t * T;
        const int n_e = (int)min((int64_t)T, e_end - e0);
        if (lane < n_e) rcv = p.identity ? (int)(e0 + lane) : p.receivers[e0 + lane];
        if (p.vec) {
            if (lane < n_e) {
#pragma unroll
                for (int i = 0; i < 3; ++i) vv[i] = p.vec[(e0 + lane) * 3 + i];
            }
            return;
        }
#pragma unroll
        for (int i = 0; i < YPL; ++i) {
            const int idx = i * 32 + lane;
            if (idx < n_e * Tab::DSH) yv[i] = p.sh[e0 * Tab::DSH + idx];
        }
    }
    // receiver ids, the "receiver changes here" bit mask, harmonics and the A entries of tile t
    __device__ __forceinline__ void fill(int t, unsigned char* st) {
        const int64_t e0 = e_begin + (int64_t)t * T;
        const int n_e = (int)min((int64_t)T, e_end - e0);
        int* recv_t = reinterpret_cast<int*>(st + L::st_r);
        float* y_t = reinterpret_cast<float*>(st + L::st_y);
        int before = __shfl_up_sync(0xffffffffu, rcv_a, 1);
        if (lane == 0) before = last_rcv;
        const unsigned mask = __ballot_sync(0xffffffffu, lane < n_e && rcv_a != before);
        last_rcv = __shfl_sync(0xffffffffu, rcv_a, n_e - 1);
        if (lane < n_e) recv_t[lane] = rcv_a;
        if (lane == 0) recv_t[T] = (int)mask;
        if (p.vec) {   // harmonics of the edge direction, formed here
            if (lane < n_e) {
                float ux, uy, uz, inv_r, Y[Tab::DSH];
                unit_vector(v_a[0], v_a[1], v_a[2], ux, uy, uz, inv_r);
                harmonics<Tab::DSH>(ux, uy, uz, Y);
#pragma unroll
                for (int i = 0; i < Tab::DSH; ++i) y_t[lane * Tab::DSH + i] = Y[i];
            }
        } else {
#pragma unroll
            for (int i = 0; i < YPL; ++i) {
                const int idx = i * 32 + lane;
                if (idx < n_e * Tab::DSH) y_t[idx] = y_a[i];
            }
        }
        if constexpr (L::DBL) {
            float* uy_t = reinterpret_cast<float*>(st + L::st_uy);
#pragma unroll
            for (int i = 0; i < YPL; ++i) {
                const int idx = i * 32 + lane;
                if (idx < n_e * Tab::DSH) uy_t[idx] = uy_a[i];
            }
        }
        __syncwarp();
        // A[e][slot] = sum over the slot's records of c * y[e][i2]: contracted once per edge here, so that
        // the consumers' per-channel loop never touches a coefficient.  All loads come before the first
        // store, so that they are in flight together.
        // (entries of edges beyond n_e are computed from stale data and never read)
        float* A_t = reinterpret_cast<float*>(st + L::st_A);
        float a_val[NA][T];
#pragma unroll
        for (int i = 0; i < NA; ++i)
#pragma unroll
            for (int e_i = 0; e_i < T; ++e_i) {
                const float* ye = y_t + e_i * Tab::DSH;
                a_val[i][e_i] = fmaf(tab[i].c1, ye[tab[i].i2_1], tab[i].c0 * ye[tab[i].i2_0]);
            }
#pragma unroll
        for (int i = 0; i < NA; ++i) {
            const int slot = lane + 32 * i;
            if (slot < Tab::APAD) {
#pragma unroll
                for (int e_i = 0; e_i < T; ++e_i) A_t[e_i * Tab::APAD + slot] = a_val[i][e_i];
            }
        }
        if constexpr (L::DBL) {   // the same contraction with the cotangent of the harmonics: B
            float* B_t = reinterpret_cast<float*>(st + L::st_B);
            const float* uy_t = reinterpret_cast<const float*>(st + L::st_uy);
#pragma unroll
            for (int i = 0; i < NA; ++i)
#pragma unroll
                for (int e_i = 0; e_i < T; ++e_i) {
                    const float* ye = uy_t + e_i * Tab::DSH;
                    a_val[i][e_i] = fmaf(tab[i].c1, ye[tab[i].i2_1], tab[i].c0 * ye[tab[i].i2_0]);
                }
#pragma unroll
            for (int i = 0; i < NA; ++i) {
                const int slot = lane + 32 * i;
                if (slot < Tab::APAD) {
#pragma unroll
                    for (int e_i = 0; e_i < T; ++e_i) B_t[e_i * Tab::APAD + slot] = a_val[i][e_i];
                }
            }
        }
        __syncwarp();
        rcv_a = rcv_b;
#pragma unroll
        for (int i = 0; i < YPL; ++i) y_a[i] = y_b[i];
#pragma unroll
        for (int i = 0; i < 3; ++i) v_a[i] = v_b[i];
        load(t + 2, rcv_b, y_b, v_b);
        if constexpr (L::DBL) {
#pragma unroll
            for (int i = 0; i < YPL; ++i) uy_a[i] = uy_b[i];
            load_ct(t + 2, uy_b);
        }
    }
};

// Lets copies that are still in flight land before the CTA's shared memory is released (abort path only).
template <class L>
__device__ __forceinline__ void drain_copies(unsigned char* smem, int armed) {
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    for (int t = max(0, armed - L::NS); t < armed; ++t)
#pragma unroll 1
        for (uint32_t it = 0; it < kSpinLimit; ++it)
            if (mbar_try_wait(&full[t % L::NS], (t / L::NS) & 1)) break;
}

// ------------------------------------------------------------------------ the producer warps
// ROLE: 0 = copies only, 1 = tables only, 2 = both (one warp).  The ring's `full` barriers expect two arrivals
// (one with the copies' byte count, one after the tables) plus the copies' bytes.
template <class L, class Tab, int ROLE, class P>
__device__ __forceinline__ void producer_loop(const P& p, unsigned char* smem, const int lane, const int64_t e_begin,
                                              const int64_t e_end, const int n_tiles) {
    constexpr int NS = L::NS;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    int armed = 0, stage = 0, phase = 0;
    if constexpr (ROLE == 0) {
        CopyPart<L, P> cp(p, lane, e_begin, e_end, n_tiles);
#pragma unroll 1
        for (int t = 0; t < n_tiles; ++t) {
            // phase of `empty` that ends the previous use of this ring slot
            if (t >= NS && !mbar_wait(&empty[stage], phase ^ 1, abort_flag, p.status)) break;
            cp.issue(t, smem + L::off_stage + stage * (int)L::stage_bytes, &full[stage]);
            armed = t + 1;
            if (++stage == NS) { stage = 0; phase ^= 1; }
        }
        if (*abort_flag) drain_copies<L>(smem, armed);
    } else if constexpr (ROLE == 1) {
        TablePart<L, Tab, P> tp(p, lane, e_begin, e_end, n_tiles);
#pragma unroll 1
        for (int t = 0; t < n_tiles; ++t) {
            if (t >= NS && !mbar_wait(&empty[stage], phase ^ 1, abort_flag, p.status)) break;
            tp.fill(t, smem + L::off_stage + stage * (int)L::stage_bytes);
            if (lane == 0) mbar_arrive(&full[stage]);  // the staged A entries and receiver ids are in place
            if (++stage == NS) { stage = 0; phase ^= 1; }
        }
    } else {
        CopyPart<L, P> cp(p, lane, e_begin, e_end, n_tiles);
        TablePart<L, Tab, P> tp(p, lane, e_begin, e_end, n_tiles);
#pragma unroll 1
        for (int t = 0; t < n_tiles; ++t) {
            if (t >= NS && !mbar_wait(&empty[stage], phase ^ 1, abort_flag, p.status)) break;
            unsigned char* st = smem + L::off_stage + stage * (int)L::stage_bytes;
            cp.issue(t, st, &full[stage]);  // copies first: they are the long pole
            armed = t + 1;
            tp.fill(t, st);
            if (lane == 0) mbar_arrive(&full[stage]);
            if (++stage == NS) { stage = 0; phase ^= 1; }
        }
        if (*abort_flag) drain_copies<L>(smem, armed);
    }
}

}  // namespace fast
}  // namespace e3j
