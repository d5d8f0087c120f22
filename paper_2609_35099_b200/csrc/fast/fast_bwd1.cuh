// Edge-wise backward pass 1: one consumer warp computes the whole backward of one edge.
//
// The path-group kernel of fast_bwd.cuh keeps each warp's rows of grad_out[receiver] in registers and pays for
// it with an exchange of partial sums between the warps after every edge.  Here the receiver's row block is
// staged once in shared memory and every warp reads the rows where its body needs them: a warp owns an edge
// from the first load to the last store, nothing is exchanged, the lane reduction of grad_sh happens once per
// edge instead of once per edge and path group, and all warps of an SM run the same instructions.
//
// Ring: NS tiles of up to T edges (T = number of consumer warps, warp j takes edge j of the tile).  A tile
// holds the edges of at most two neighbouring receivers (one in the fused double backward), so that the last
// tile of a receiver is filled up with the first edges of the next one instead of leaving warps idle; the
// staged row blocks of grad_out form a ring of their own (three for two receivers per tile, NS for one) that
// advances when the receiver changes.  With NS = 2 tiles in flight a new receiver's block must not be one that
// the tile before reads: three blocks allow that as long as a tile that starts a new receiver right after a
// two-receiver tile stays with that one receiver (graphs with one or two edges per receiver).
// The producer warp cuts the tiles, issues the bulk copies (weights, sender rows, the receiver's block when
// it is new) and contracts the A entries; the metadata it needs (receiver and sender ids, harmonics) arrives
// two 32-edge windows ahead through 4-byte asynchronous copies.
//
// Standalone tensor product (ROWS = true): every row is its own sender and receiver, so its grad_out block
// travels with it in the ring slot, tiles are fixed runs of T rows, and each ring slot has its own T consumer
// warps (a slot of a 100-row signature is 70 KB: three of them, one warp each, keep more bytes in flight than
// a double-buffered pair would).
//
// Fused double backward (DBL = true, graph calls): the same sweep with the cotangents (ux, uy, us) of
// (grad_x, grad_sh, grad_w) staged beside (x, y, s) -- two sender rows, two weight rows and two A tables per
// edge -- and the body S::bwd2_edge_all, which yields the cotangents of s and y and this edge's share of the
// cotangent of x (the message-passing double backward of the paper, its three edge outputs; the cotangent of
// grad_out is a forward-shaped sum and has its own kernel).
//
// Channels beyond one warp's (CH = N_q / (32 EV) > 1): CH warps share an edge, each with its own channels.
// Only the channel sum of grad_sh joins them: every warp leaves its 16 partial sums in the slot, and the first
// warp of the edge adds them in warp order once all have arrived (bounded wait on a barrier of their own).
#pragma once
#include "fast_bwd.cuh"
#include "fast_producer.cuh"

namespace e3j {
namespace fast {

__device__ __forceinline__ void cp_async4(void* dst_smem, const void* src_gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst_smem)), "l"(src_gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <class S, bool ROWS, bool DBL = false>
struct Bwd1Smem {
    static_assert(!(ROWS && DBL), "the fused double backward exists for graph calls only");
    static constexpr int T = DBL ? S::DT : ROWS ? S::ETR : S::ET, NS = DBL ? S::DS : ROWS ? S::ESR : S::ES;
    static constexpr int VW = DBL ? S::DV : S::EV;  // channels per lane
    using Vec = typename VecOf<VW>::type;
    static constexpr int CH = S::NQ / (32 * VW);    // warps per edge
    static constexpr int NG = ROWS ? NS : 1;        // groups of T * CH consumer warps (ROWS: one per ring slot)
    static constexpr int S_EDGE = S::P * S::NQ;
    static constexpr int X_EDGE = S::DIN * S::NQ;
    static constexpr int DM_ROW = S::D * S::NQ;     // grad_out[receiver]
    static constexpr int WIN = 32;                  // edges per metadata window; the ring holds two windows
    static constexpr size_t up(size_t v, size_t a) { return (v + a - 1) / a * a; }
    static constexpr size_t off_bar = 0;                                   // full[NS], empty[NS]
    static constexpr size_t off_join = off_bar + 16 * NS;                  // join[NS][T]: the CH warps of an edge
    static constexpr size_t off_abort = off_join + 8 * NS * T;
    static constexpr size_t off_meta = up(off_abort + 4, 16);              // int[NS][4]: first edge, n_e | last << 8, block a | block b << 8 | edges of a << 16
    static constexpr size_t off_rcv = off_meta + 16 * NS;                  // int[2 * WIN]
    static constexpr size_t off_snd = off_rcv + 4 * 2 * WIN;               // int[2 * WIN]
    static constexpr size_t off_y = off_snd + 4 * 2 * WIN;                 // float[2 * WIN][DSH]
    static constexpr size_t off_uy = off_y + 4 * 2 * WIN * S::DSH;         // float[2 * WIN][DSH] (DBL)
    static constexpr size_t off_dm = up(off_uy + (DBL ? 4 * 2 * WIN * S::DSH : 0), 128);  // float[NS][D][NQ] (graph calls)
    static constexpr int NIN = DBL ? 2 : 1;         // copies of every per-edge input (DBL: primal and cotangent)
    static constexpr size_t st_s = 0;
    static constexpr size_t st_us = st_s + 4 * (size_t)T * S_EDGE;               // (DBL)
    static constexpr size_t st_x = st_s + 4 * (size_t)NIN * T * S_EDGE;
    static constexpr size_t st_ux = st_x + 4 * (size_t)T * X_EDGE;               // (DBL)
    static constexpr size_t st_A = st_x + 4 * (size_t)NIN * T * X_EDGE;
    static constexpr size_t st_B = st_A + 4 * (size_t)T * S::B_APAD;             // (DBL)
    static constexpr size_t st_dy = st_A + 4 * (size_t)NIN * T * S::B_APAD;      // float[T][CH][16] (CH > 1)
    static constexpr size_t st_dm = up(st_dy + (CH > 1 ? 4 * (size_t)T * CH * 16 : 0), 128);   // float[T][D][NQ] (ROWS)
    static constexpr size_t stage_bytes = up(st_dm + (ROWS ? 4 * (size_t)T * DM_ROW : 0), 128);
    // Receivers a tile may hold and staged grad_out row blocks: two receivers per tile need three blocks (see the
    // head of this file); signatures whose rows are too large for a third block keep one receiver per tile.
    static constexpr size_t total_with(int nd) {
        return up(off_dm + (ROWS ? 0 : 4 * (size_t)nd * DM_ROW), 128) + NS * stage_bytes;
    }
    static constexpr int MAXR = (!ROWS && !DBL && NS == 2 && T < 29 && total_with(3) + 1024 <= 228 * 1024) ? 2 : 1;
    static constexpr int ND = MAXR == 2 ? 3 : NS;
    static constexpr size_t off_stage = up(off_dm + (ROWS ? 0 : 4 * (size_t)ND * DM_ROW), 128);
    static constexpr size_t total = off_stage + NS * stage_bytes;
};

// ------------------------------------------------------------------------ consumer: one edge per tile
template <class S, bool ROWS, bool DBL>
__device__ __forceinline__ void bwd1_consumer(const BwdParams& p, unsigned char* smem, const int warp, const int lane,
                                              const int64_t e_begin, const int64_t e_end) {
    using L = Bwd1Smem<S, ROWS, DBL>;
    using Vec = typename L::Vec;
    constexpr int NS = L::NS, VW = L::VW;
    constexpr int NQV = S::NQ / VW;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    constexpr int CH = L::CH;
    const int j = (warp / CH) % L::T;            // this warp's edge of a tile
    const int c = warp % CH;                     // and its share of the channels
    const int vlane = c * 32 + lane;
    uint64_t* join = reinterpret_cast<uint64_t*>(smem + L::off_join);
    int stage = ROWS ? warp / (L::T * CH) : 0, phase = 0;
    unsigned join_phase = 0;   // bit s: parity of the next use of this edge slot's join barrier in ring slot s
    // ROWS: tiles are fixed runs of T rows and this warp's group takes every NS-th of them
    int my_tiles = ROWS ? ((int)((e_end - e_begin + L::T - 1) / L::T) - stage + NS - 1) / NS : 1;
    while (my_tiles > 0) {
        if (!mbar_wait(&full[stage], phase, abort_flag, p.status)) break;
        const int* meta = reinterpret_cast<const int*>(smem + L::off_meta) + 4 * stage;
        const int first = meta[0], n_e = meta[1] & 0xff, last = meta[1] >> 8;
        const int block = j < (meta[2] >> 16) ? (meta[2] & 0xff) : ((meta[2] >> 8) & 0xff);   // this edge's receiver
        if (j < n_e) {
            const unsigned char* st = smem + L::off_stage + stage * (int)L::stage_bytes;
            const int64_t e = e_begin + first + j;
            const Vec* xs = reinterpret_cast<const Vec*>(st + L::st_x) + j * (L::X_EDGE / VW) + vlane;
            const Vec* ss = reinterpret_cast<const Vec*>(st + L::st_s) + j * (L::S_EDGE / VW) + vlane;
            const float* As = reinterpret_cast<const float*>(st + L::st_A) + j * S::B_APAD;
            const Vec* dms = (ROWS ? reinterpret_cast<const Vec*>(st + L::st_dm) + j * (L::DM_ROW / VW)
                                   : reinterpret_cast<const Vec*>(smem + L::off_dm + (size_t)block * 4 * L::DM_ROW)) + vlane;
            Vec dxp[S::DIN];   // both are assigned (not accumulated into) by bwd_edge_all
            float dyl[16];
            Vec* gw = p.grad_w ? reinterpret_cast<Vec*>(p.grad_w + (size_t)e * L::S_EDGE) + vlane : nullptr;   // null: not wanted
            if constexpr (DBL) {
                const Vec* uxs = reinterpret_cast<const Vec*>(st + L::st_ux) + j * (L::X_EDGE / VW) + vlane;
                const Vec* uss = reinterpret_cast<const Vec*>(st + L::st_us) + j * (L::S_EDGE / VW) + vlane;
                const float* Bs = reinterpret_cast<const float*>(st + L::st_B) + j * S::B_APAD;
                S::bwd2_edge_all(dms, xs, uxs, ss, uss, As, Bs, dxp, dyl, gw);
            } else {
                S::bwd_edge_all(dms, xs, ss, As, dxp, dyl, gw);
            }
            Vec* dxo = reinterpret_cast<Vec*>(p.dx_edge + (size_t)e * L::X_EDGE) + vlane;
#pragma unroll
            for (int i = 0; i < S::DIN; ++i) dxo[i * NQV] = dxp[i];
            // sum over the channels: even lanes end up with one entry each
            const float dy_tot = reduce16_over_lanes(dyl, lane);
            const int idx = ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
            if constexpr (CH == 1) {
                if ((lane & 1) == 0 && idx < S::DSH && p.grad_sh) p.grad_sh[(size_t)e * S::DSH + idx] = dy_tot;
            } else {
                float* dyx = const_cast<float*>(reinterpret_cast<const float*>(st + L::st_dy)) + j * CH * 16;
                if ((lane & 1) == 0) dyx[c * 16 + idx] = dy_tot;
                __syncwarp();
                if (lane == 0) mbar_arrive(&join[stage * L::T + j]);
                if (c == 0) {   // fixed-order sum over the edge's warps
                    if (!mbar_wait(&join[stage * L::T + j], (join_phase >> stage) & 1u, abort_flag, p.status)) break;
                    if (lane < S::DSH) {
                        float sum = 0.f;
#pragma unroll
                        for (int c2 = 0; c2 < CH; ++c2) sum += dyx[c2 * 16 + lane];
                        if (p.grad_sh) p.grad_sh[(size_t)e * S::DSH + lane] = sum;
                    }
                }
                join_phase ^= 1u << stage;   // (a short tile leaves the barriers of its unused edge slots alone)
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[stage]);
        if (ROWS) {
            phase ^= 1;   // this group's slot again, one trip round the ring later
            --my_tiles;
        } else {
            if (++stage == NS) { stage = 0; phase ^= 1; }
            if (last) break;
        }
    }
}

// ------------------------------------------------------------------------ producer
template <class S, bool ROWS, bool DBL>
__device__ __forceinline__ void bwd1_producer(const BwdParams& p, unsigned char* smem, const int lane,
                                              const int64_t e_begin, const int64_t e_end) {
    using L = Bwd1Smem<S, ROWS, DBL>;
    using Tab = BwdTab<S>;
    constexpr int T = L::T, NS = L::NS, WIN = L::WIN, DSH = S::DSH;
    constexpr int NA = (Tab::APAD + 31) / 32;
    static_assert(T < 32 && WIN == 32, "a tile is cut with one ballot; windows are one warp wide");
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);
    int* rcv_ring = reinterpret_cast<int*>(smem + L::off_rcv);
    int* snd_ring = reinterpret_cast<int*>(smem + L::off_snd);
    float* y_ring = reinterpret_cast<float*>(smem + L::off_y);
    float* uy_ring = reinterpret_cast<float*>(smem + L::off_uy);
    const int n_tot = (int)(e_end - e_begin);

    ASlot tab[NA];   // this lane's A slots (lane, lane + 32, ...)
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

    // window w = edges [32 w, 32 w + 32) of this CTA's range, kept in ring half (w & 1); one copy group each
    auto issue_window = [&](const int w) {
        const int i = WIN * w + lane;
        const int half = (w & 1) * WIN;
        if (!ROWS && i < n_tot) {
            cp_async4(&rcv_ring[half + lane], p.receivers + e_begin + i);
            cp_async4(&snd_ring[half + lane], p.senders + e_begin + i);
        }
#pragma unroll
        for (int j = 0; j < DSH; ++j) {
            const int idx = j * 32 + lane;   // entry of the window's [32][DSH] block
            if (WIN * w + idx / DSH < n_tot) {
                cp_async4(&y_ring[half * DSH + idx], p.sh + (e_begin + (int64_t)WIN * w) * DSH + idx);
                if (DBL) cp_async4(&uy_ring[half * DSH + idx], p.ct_sh + (e_begin + (int64_t)WIN * w) * DSH + idx);
            }
        }
        cp_async_commit();
    };
    issue_window(0);
    issue_window(1);

    if (ROWS && n_tot == 0) {    // the consumers of a call without rows expect no tile
        cp_async_wait<0>();
        return;
    }
    int wbase = 0;               // windows wbase and wbase + 1 are in the ring or on their way
    int done = 0;                // edges handed out so far
    int block = L::ND - 1;       // ring position of the current receiver's grad_out block
    bool prev_second = false;    // the tile before held edges of two receivers
    int last_rcv = -1;
    int stage = 0, phase = 0, armed = 0;
#pragma unroll 1
    for (int t = 0;; ++t) {
        if ((done >> 5) > wbase) {   // the half that held window wbase - 1 is free
            wbase = done >> 5;
            issue_window(wbase + 1);
        }
        // the newest group may stay in flight unless this tile reaches into it
        if ((done & 31) + T > WIN) cp_async_wait<0>(); else cp_async_wait<1>();
        __syncwarp();
        // the tile: edges done .. done + n_e - 1 of at most MAXR receivers (ROWS: the next T rows)
        const int i = done + lane;
        int r0 = -1, r1 = -1, n_e, n_a = 0;   // n_a: edges of the first receiver
        if (ROWS) {
            n_e = min(T, n_tot - done);
        } else {
            const int r = (lane < T && i < n_tot) ? rcv_ring[i & (2 * WIN - 1)] : -2;
            r0 = __shfl_sync(0xffffffffu, r, 0);
            const unsigned differs = __ballot_sync(0xffffffffu, r != r0);   // lane T always differs
            n_a = n_tot > 0 ? __ffs((int)differs) - 1 : 0;
            n_e = n_a;
            // fill up with the next receiver's edges -- unless that receiver's row block would land on one that the
            // tile before (still in flight) reads: the case when that tile held two receivers and this one starts a third
            if (L::MAXR == 2 && n_a > 0 && n_a < T && done + n_a < n_tot && !(prev_second && r0 != last_rcv)) {
                r1 = __shfl_sync(0xffffffffu, r, n_a);
                const unsigned differs2 = __ballot_sync(0xffffffffu, lane >= n_a && r != r1);
                n_e = __ffs((int)differs2) - 1;
            }
        }
        const int last = done + n_e >= n_tot;
        // phase of `empty` that ends the previous use of this ring slot
        if (t >= NS && !mbar_wait(&empty[stage], phase ^ 1, abort_flag, p.status)) break;
        const bool new_block = !ROWS && n_e > 0 && r0 != last_rcv;
        if (new_block) {
            block = block + 1 == L::ND ? 0 : block + 1;
            last_rcv = r0;
        }
        const int block_a = block;
        const bool second = r1 >= 0;   // the tile goes on into the next receiver: its block is new by definition
        if (second) {
            block = block + 1 == L::ND ? 0 : block + 1;
            last_rcv = r1;
        }
        prev_second = second;
        unsigned char* st = smem + L::off_stage + stage * (int)L::stage_bytes;
        if (lane == 0) {
            int* meta = reinterpret_cast<int*>(smem + L::off_meta) + 4 * stage;
            meta[0] = done; meta[1] = n_e | (last << 8); meta[2] = block_a | (block << 8) | (n_a << 16);
            // arrival and byte count in one step: the phase cannot complete before the bytes are expected
            mbar_arrive_expect_tx(&full[stage], (uint32_t)n_e * 4u * (L::NIN * (L::S_EDGE + L::X_EDGE) + (ROWS ? L::DM_ROW : 0)) +
                                                    ((new_block ? 4u : 0u) + (second ? 4u : 0u)) * L::DM_ROW);
            if (n_e > 0)
                bulk_g2s(st + L::st_s, p.w + (size_t)(e_begin + done) * L::S_EDGE, (uint32_t)n_e * 4u * L::S_EDGE,
                         &full[stage]);
        }
        if (ROWS) {   // the rows' inputs and grad_out blocks are contiguous
            if (lane == 1)
                bulk_g2s(st + L::st_x, p.x + (size_t)(e_begin + done) * L::X_EDGE, (uint32_t)n_e * 4u * L::X_EDGE,
                         &full[stage]);
            if (lane == 2)
                bulk_g2s(st + L::st_dm, p.grad_out + (size_t)(e_begin + done) * L::DM_ROW,
                         (uint32_t)n_e * 4u * L::DM_ROW, &full[stage]);
        } else {
            if (lane < n_e) {
                const size_t snd = (size_t)snd_ring[i & (2 * WIN - 1)];
                bulk_g2s(st + L::st_x + (size_t)lane * 4 * L::X_EDGE, p.x + snd * L::X_EDGE, 4u * L::X_EDGE, &full[stage]);
                if (DBL)
                    bulk_g2s(st + L::st_ux + (size_t)lane * 4 * L::X_EDGE, p.ct_x + snd * L::X_EDGE, 4u * L::X_EDGE,
                             &full[stage]);
            }
            if (DBL && lane == 30 && n_e > 0)
                bulk_g2s(st + L::st_us, p.ct_w + (size_t)(e_begin + done) * L::S_EDGE, (uint32_t)n_e * 4u * L::S_EDGE,
                         &full[stage]);
            if (lane == 29 && second)
                bulk_g2s(smem + L::off_dm + (size_t)block * 4 * L::DM_ROW, p.grad_out + (size_t)r1 * L::DM_ROW,
                         4u * L::DM_ROW, &full[stage]);
            if (lane == 31 && new_block)
                bulk_g2s(smem + L::off_dm + (size_t)block_a * 4 * L::DM_ROW, p.grad_out + (size_t)r0 * L::DM_ROW,
                         4u * L::DM_ROW, &full[stage]);
        }
        armed = t + 1;
        // A[e][slot] = sum over the slot's records of c * y[e][i2]; all loads before the first store
        // (entries of edges beyond n_e are computed from stale data and never read)
#pragma unroll
        for (int tbl = 0; tbl < L::NIN; ++tbl) {   // A from the harmonics; DBL: B from their cotangent as well
            float* A_t = reinterpret_cast<float*>(st + (tbl ? L::st_B : L::st_A));
            const float* ring = tbl ? uy_ring : y_ring;
            float a_val[NA][T];
#pragma unroll
            for (int k = 0; k < NA; ++k)
#pragma unroll
                for (int e_i = 0; e_i < T; ++e_i) {
                    const float* ye = ring + ((done + e_i) & (2 * WIN - 1)) * DSH;
                    a_val[k][e_i] = fmaf(tab[k].c1, ye[tab[k].i2_1], tab[k].c0 * ye[tab[k].i2_0]);
                }
#pragma unroll
            for (int k = 0; k < NA; ++k) {
                const int slot = lane + 32 * k;
                if (slot < Tab::APAD) {
#pragma unroll
                    for (int e_i = 0; e_i < T; ++e_i) A_t[e_i * Tab::APAD + slot] = a_val[k][e_i];
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&full[stage]);   // the staged A entries and the tile's metadata are in place
        if (++stage == NS) { stage = 0; phase ^= 1; }
        done += n_e;
        if (last) break;
    }
    cp_async_wait<0>();
    if (*abort_flag) drain_copies<L>(smem, armed);
}

template <class S, bool ROWS, bool DBL = false>
__global__ void __launch_bounds__((Bwd1Smem<S, ROWS, DBL>::T * Bwd1Smem<S, ROWS, DBL>::CH * Bwd1Smem<S, ROWS, DBL>::NG + 1) * 32, 1)
fast_bwd1_kernel(const BwdParams p) {
    using L = Bwd1Smem<S, ROWS, DBL>;
    constexpr int T = L::T, NS = L::NS, NCONS = L::T * L::CH * L::NG;
    static_assert(S::NQ == 32 * L::VW * L::CH, "the channels are dealt out to whole warps");
    static_assert(S::B_NREC <= 2, "an A slot holds at most two records");
    static_assert(S::DSH <= 16, "harmonics beyond l = 3 need a wider reduction");

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::off_bar);
    uint64_t* empty = full + NS;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::off_abort);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int64_t n_edges, chunk, e_begin, e_end;   // n_edges: the real edges (a padded call learns their number here)
    cta_edge_range(p.n_edges, p.chunk, p.n_real, n_edges, chunk, e_begin, e_end);

    if (threadIdx.x == 0) {
        // full: the producer's arrival with the copies' byte count and its arrival after the tables;
        // empty: the T warps that work on the slot
        for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 2); mbar_init(&empty[s], T * L::CH); }
        for (int s = 0; s < NS * T; ++s) mbar_init(reinterpret_cast<uint64_t*>(smem + L::off_join) + s, L::CH);
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    if (warp == NCONS) bwd1_producer<S, ROWS, DBL>(p, smem, lane, e_begin, e_end);
    else bwd1_consumer<S, ROWS, DBL>(p, smem, warp, lane, e_begin, e_end);
}

}  // namespace fast
}  // namespace e3j
