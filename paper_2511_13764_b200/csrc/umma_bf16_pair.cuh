// BF16 GEMM on CTA pairs: two CTAs (a cluster of 2, neighbouring SMs) compute one
// 256 x BN output tile with a single tcgen05.mma.cta_group::2 per k-step.
//
// Why: with one CTA per tile every SM has to pull 128 rows of A and BN columns of B per
// k-block from L2, and that operand feed, not the tensor pipe, bounds the single-CTA
// kernel.  In a pair each CTA loads its own 128 rows of A and only HALF of the B tile; the
// tensor cores of both SMs read both halves.  Bytes per flop per SM drop by a third at
// BN = 256 and the freed shared memory buys two more pipeline stages.  No TMA multicast is
// used: every CTA fetches its own boxes; only the mbarrier signals cross the pair.
//
// The structure is that of the single-CTA kernel (Algorithm 1 of the paper: tile loop,
// accumulator resident over the K loop, fused epilogue, one store).  Differences:
//   - both CTAs' TMA loads complete on the LEADER's (rank 0) full[] barrier, which expects
//     the bytes of both;
//   - only the leader issues MMAs; tcgen05.commit signals empty[] and tmem_full[] in both CTAs;
//   - each CTA drains its own 128 accumulator rows; tmem_empty[] lives in the leader and
//     counts the epilogue threads of both CTAs (the peer arrives remotely);
//   - cluster-wide barriers fence the start (barriers initialised) and the end (nobody
//     leaves while its peer may still touch its shared memory or barriers).
//
// Tail mode (p.tail_from >= 0), the stream-K treatment of a ragged last wave: the tiles that are
// left after the last full wave would occupy a fraction of the pairs for a whole K loop.  Their
// k-blocks, laid end to end, are instead shared out evenly over ALL the pairs (p.sk_share each),
// so the wave takes a fraction of a K loop.  A pair's range covers part of one tile or the end
// of one and the start of the next; for each part it writes an FP32 (INT32 for INT8) partial
// slab, and a small kernel (tail_reduce_kernel) adds the slabs of a tile in segment order, which
// is k order: deterministic, no atomics.  Units 0 .. tail_from-1 are whole tiles.
//
// With CLUSTER_REDUCE the cluster holds S pairs, one per K split of the same 256-row tile
// (ranks 2s and 2s + 1 are the pair of split s; a pair's leader is its even rank); the
// accumulators of the S CTAs that own the same 128 rows are summed through distributed shared
// memory exactly as in the single-CTA kernel (umma_cluster_epilogue).
#pragma once
#include "umma_bf16.cuh"

namespace nk {

__host__ __device__ constexpr int pair_stage_bytes(int BN) { return UMMA_A_STAGE_BYTES + (BN / 2) * UMMA_BK * 2; }
__host__ __device__ constexpr int pair_smem_bytes(int BN, int stages) {
    return stages * pair_stage_bytes(BN) + 1024 + UMMA_EPI_STAGING + 384;
}

// UmmaParams as for the single-CTA kernel, with tiles_m counted in 256-row tiles.
template <int BN, int STAGES, bool B_VNNI, bool CLUSTER_REDUCE = false, int KIND = 0>
__global__ void __launch_bounds__(UMMA_THREADS, 1)
umma_bf16_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                      const __grid_constant__ CUtensorMap tmap_c, const UmmaParams p) {
    static_assert(BN == 128 || BN == 256, "pair tile N");
    constexpr int HALF = BN / 2;                       // B columns held by each CTA
    constexpr int B_STAGE = HALF * UMMA_BK * 2;
    constexpr int STAGE = pair_stage_bytes(BN);
    constexpr uint32_t TMEM_COLS = 2 * BN;             // two accumulators of BN columns
    constexpr int BM2 = 2 * UMMA_BM;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar_base = smem_base + STAGES * STAGE + UMMA_EPI_STAGING;   // stages, epilogue staging, barriers
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
    auto raw_bar = [&](int s) { return bar_base + UMMA_RAW_BAR_OFFSET + 8u * s; };   // VNNI B: this CTA's blocks of stage s have landed
    const uint32_t peer_ready_bar = bar_base + 192u;   // leader: the peer CTA has allocated its tensor memory
    const uint32_t recv_bar0 = bar_base + UMMA_RECV_BAR_OFFSET;   // cluster split-K: pieces for epilogue warp w have landed
    uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
    volatile uint32_t* tmem_slot =
        reinterpret_cast<volatile uint32_t*>(gen_base + STAGES * STAGE + UMMA_EPI_STAGING + 8 * (2 * STAGES + 4));
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t crank = cluster_ctarank();          // rank in the cluster (0, 1 unless CLUSTER_REDUCE)
    const uint32_t rank = crank & 1u;                  // half of the pair: 0 = leader
    const uint32_t leader = crank & ~1u;               // cluster rank of this pair's leader
    const uint16_t pair_mask = static_cast<uint16_t>(3u << leader);   // both CTAs of this pair
    const int pair_id = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;

    if (warp == 0) {
        // one barrier per lane: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2] (and raw[STAGES]).
        // full[]: the leader's producer (+ the 2 re-layout warps per CTA whose turn the stage is); tmem_empty[]: the epilogue threads of both CTAs
        constexpr int NB = 2 * STAGES + 4;
        static_assert(NB <= 32, "one barrier per lane");
        static_assert(!B_VNNI || STAGES % 2 == 0, "the re-layout warps take alternate stages");
        if (lane < NB)
            mbar_init(bar_base + 8u * lane, lane < STAGES ? (B_VNNI ? 1 + 4 : 1) : lane < 2 * STAGES + 2 ? 1 : 256);
        if (B_VNNI && lane < STAGES) mbar_init(raw_bar(lane), 1);
        if (lane == 31) mbar_init(peer_ready_bar, 1);
        if (CLUSTER_REDUCE && lane >= 20 && lane < 28) mbar_init(recv_bar0 + 8u * (lane - 20), 1);   // one per epilogue warp
        if (lane == 0) *abort_flag = 0;
        fence_mbar_init();
        __syncwarp();
    } else if (warp == 2 && lane == 0) {
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
        if (p.tma_store) tma_prefetch_desc(&tmap_c);
    }
    // Start-up.  Every thread arrives on the cluster barrier at once (warp 0 after its barriers
    // are initialised: the arrive releases them to the other CTAs) and waits on it before it first
    // touches a barrier of the peer; the tensor-memory allocation runs meanwhile, and the producer
    // starts fetching without waiting for it.  What the leader's MMA warp needs besides is the
    // PEER's allocation: the peer's warp 1 reports it on the leader's `peer_ready` barrier.
    cluster_arrive();
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
        tmem_relinquish_pair();
    }
    const uint32_t nthreads = blockDim.x;
    uint32_t tmem_base = 0;
    if (warp == 0) {
        cluster_wait();
        asm volatile("bar.arrive 0, %0;" ::"r"(nthreads) : "memory");
    } else {
        tc_fence_before_sync();
        cluster_wait();
        if (warp == 1 && rank == 1 && lane == 0) mbar_arrive_cluster_cta_release(map_to_cta(peer_ready_bar, leader));
        asm volatile("bar.sync 0, %0;" ::"r"(nthreads) : "memory");
        tc_fence_after_sync();
        tmem_base = *tmem_slot;
    }

    const bool tail_mode = p.tail_from >= 0;
    // tail mode: every pair has its whole tiles (units below tail_from, a multiple of the number of
    // pairs) and then up to two segments of the tail (its k-block range may straddle two tiles)
    const int total_units = tail_mode ? p.tail_from + 2 * num_pairs : p.gemms * p.tiles_m * p.tiles_n * p.splits;
    // unit -> tile, K split (segment number inside a tail tile), GEMM of the batch, k-block range;
    // tail >= 0: index of the tail tile.  False: nothing to do (an empty segment; only a pair's last
    // units can be empty, so the accumulator and barrier phases of the roles stay in step).
    auto decode = [&](int unit, int& tile, int& split, int& gemm, int& kb0, int& kb1, int& tail) -> bool {
        tail = -1;
        if (tail_mode) {
            gemm = 0;
            if (unit < p.tail_from) {
                tile = unit; split = 0; kb0 = 0; kb1 = p.kb_total;
                return true;
            }
            const int u = unit - p.tail_from;
            const int second = u >= num_pairs ? 1 : 0;
            const int j = u - second * num_pairs;                       // this pair
            const int total = (p.tiles_m * p.tiles_n - p.tail_from) * p.kb_total;
            const int start = j * p.sk_share, end = min(start + p.sk_share, total);
            if (start >= end) return false;
            const int first_tile = div_small(start, p.kb_total);
            if (!second) {
                tail = first_tile;
                kb0 = start - first_tile * p.kb_total;
                kb1 = min(p.kb_total, end - first_tile * p.kb_total);
            } else {
                tail = first_tile + 1;
                kb0 = 0;
                kb1 = end - tail * p.kb_total;
                if (kb1 <= 0) return false;
            }
            tile = p.tail_from + tail;
            split = j - div_small(tail * p.kb_total, p.sk_share);       // segments of a tile are numbered by pair
            return true;
        }
        umma_decode_unit(p, unit, tile, split, gemm);
        kb0 = split * p.kb_per_split;
        kb1 = min(p.kb_total, kb0 + p.kb_per_split);
        return true;
    };
    // a pair with a single tile to deliver, stored by TMA: its epilogue is batched through the idle ring
    const bool one_shot = !CLUSTER_REDUCE && p.tma_store && p.splits == 1 && !tail_mode && total_units <= num_pairs;
    auto give_up = [&](unsigned int code) {
        *abort_flag = 1;
        if (p.status) atomicCAS(p.status, 0u, code);
    };

    if (warp == 0) {
        // ------------------------------------------------ TMA producer (both CTAs)
        const bool a_blk = p.a_blocked != 0;
        const bool b3d = p.b_3d != 0;
        const bool b_kmajor = p.b_kmajor != 0;
        const uint32_t lead_full0 = map_to_cta(full_bar(0), leader);  // leader's full[0], cluster address
        const uint32_t elected = elect_one();
        const uint32_t lead_elected = rank == 0 ? elected : 0u;      // only the leader's barrier expects the bytes
        int stage = 0;
        uint32_t phase = 0;
        uint32_t sa = smem_base, fb = full_bar(0), lfb = lead_full0;
        bool ok = true;
        int local = 0;
        for (int unit = pair_id; ok && unit < total_units; unit += num_pairs, ++local) {
            int tile, split, gemm, kb0, kb1, tail;
            if (!decode(unit, tile, split, gemm, kb0, kb1, tail)) continue;
            int mb, nb;
            umma_tile_coords(p, tile, mb, nb);
            // K order of a whole tile: downwards on a pair's odd tiles when the plan asks for it
            const bool k_down = p.k_serpentine && (local & 1) && kb0 == 0 && kb1 == p.kb_total;
            const int row0 = mb * BM2 + static_cast<int>(rank) * UMMA_BM;
            const int col0 = nb * BN + static_cast<int>(rank) * HALF;
            int item = kb0 == 0 ? 0 : div_small(kb0, p.kb_per_item);
            int kbl = kb0 - item * p.kb_per_item;
            item += gemm;   // independent batch: the unit's own (A, B) pair
            int ia, ib;
            umma_item_pair(p, item, ia, ib);
            if (k_down) kbl = kb1 - 1;
            const int kstep = k_down ? -1 : 1;
            for (int kb = kb0; kb < kb1; ++kb) {
                const int kx = kbl * (KIND != 0 ? 2 * UMMA_BK : UMMA_BK);   // 128 bytes of k per stage row
                if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) {
                    if (lane == 0) give_up(0x100u + stage);
                    ok = false;
                    break;
                }
                {
                    // issued by the elected lane; the warp stays convergent (see elect_one)
                    const uint32_t sb = sa + UMMA_A_STAGE_BYTES;
                    mbar_arrive_expect_tx_if(fb, 2u * (UMMA_A_STAGE_BYTES + (B_VNNI ? 0 : B_STAGE)), lead_elected);
                    if (a_blk) {
                        tma_load_5d_pair_if(sa, &tmap_a, lfb, 0, 0, kbl * 2, row0 / 32, ia, elected);
                        tma_load_5d_pair_if(sa + 8192, &tmap_a, lfb, 0, 0, kbl * 2 + 1, row0 / 32, ia, elected);
                    } else {
                        tma_load_3d_pair_if(sa, &tmap_a, lfb, kx, row0, ia, elected);
                    }
                    if (B_VNNI) {
                        // this CTA's column blocks as they are, on its own barrier; its warps 6-9 re-lay them in place
                        mbar_arrive_expect_tx_if(raw_bar(stage), B_STAGE, elected);
                        tma_load_4d_if(sb, &tmap_b, raw_bar(stage), 0, kbl * (UMMA_BK / 2), col0 >> 5, ib, elected);
                    } else if (b_kmajor) {
                        tma_load_3d_pair_if(sb, &tmap_b, lfb, kx, col0, ib, elected);   // this CTA's HALF rows (n) of 128 bytes of k
                    } else {
                        if (b3d) {
                            tma_load_4d_pair_if(sb, &tmap_b, lfb, 0, kx, col0 >> 6, ib, elected);
                        } else {
#pragma unroll
                            for (int j = 0; j < HALF / 64; ++j)
                                tma_load_3d_pair_if(sb + j * 8192, &tmap_b, lfb, col0 + j * 64, kx, ib, elected);
                        }
                    }
                }
                kbl += kstep;
                if (kbl == p.kb_per_item) { kbl = 0; ++item; umma_item_pair(p, item, ia, ib); }
                __syncwarp();
                sa += STAGE;
                fb += 8;
                lfb += 8;
                if (++stage == STAGES) { stage = 0; phase ^= 1u; sa = smem_base; fb = full_bar(0); lfb = lead_full0; }
            }
        }
        if (ok) {   // drain: every stage this CTA filled has been consumed
            for (int s = 0; s < STAGES; ++s) {
                if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) break;
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (leader only)
        // Lean issue loop: see the single-CTA kernel for the descriptor layouts.  Descriptor
        // addresses are CTA-relative, so the leader's offsets name the same tiles in the peer.
        if (rank == 0) {
            const bool a_blk = p.a_blocked != 0;
            const uint64_t da0 = a_blk ? make_smem_desc(smem_base, 16, 512, 4) : make_smem_desc(smem_base, 16, 1024, 2);
            const bool b_k = B_VNNI || p.b_kmajor != 0;
            const uint64_t db0 = b_k ? make_smem_desc(smem_base + UMMA_A_STAGE_BYTES, 16, 1024, 2)
                                     : make_smem_desc(smem_base + UMMA_A_STAGE_BYTES, 8192, 1024, 2);
            const uint32_t a_hi = static_cast<uint32_t>(da0 >> 32), b_hi = static_cast<uint32_t>(db0 >> 32);
            const uint32_t a_lo0 = static_cast<uint32_t>(da0), b_lo0 = static_cast<uint32_t>(db0);
            const uint32_t a_s1 = 2u, a_s2 = a_blk ? 512u : 4u, a_s3 = a_blk ? 514u : 6u;
            const uint32_t b_s = b_k ? 2u : 128u, b_s2 = 2 * b_s, b_s3 = 3 * b_s;
            constexpr uint32_t STAGE16 = STAGE >> 4;
            const uint32_t idesc = p.idesc;
            const uint32_t elected = elect_one();
            int stage = 0;
            uint32_t phase = 0;
            uint32_t soff = 0;
            int local = 0;
            bool ok = true;
            // the MMAs write the peer's half of the accumulator: its tensor memory must be allocated
            if (!mbar_wait(peer_ready_bar, 0u, abort_flag)) {
                if (lane == 0) give_up(0x700u);
                ok = false;
            }
            for (int unit = pair_id; ok && unit < total_units; unit += num_pairs, ++local) {
                int tile, split, gemm, kb0, kb1, tail;
                if (!decode(unit, tile, split, gemm, kb0, kb1, tail)) continue;
                const int acc = local & 1;
                if (!mbar_wait(tempty_bar(acc), ((local >> 1) & 1u) ^ 1u, abort_flag)) {
                    if (lane == 0) give_up(0x200u + acc);
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * BN;
                uint32_t accumulate = 0u;
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag)) {
                        if (lane == 0) give_up(0x300u + stage);
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    {
                        const uint32_t a_lo = a_lo0 + soff, b_lo = b_lo0 + soff;
                        umma_pair_if<KIND>(d_tmem, a_lo, a_hi, b_lo, b_hi, idesc, accumulate, elected);
                        umma_pair_if<KIND>(d_tmem, a_lo + a_s1, a_hi, b_lo + b_s, b_hi, idesc, 1u, elected);
                        umma_pair_if<KIND>(d_tmem, a_lo + a_s2, a_hi, b_lo + b_s2, b_hi, idesc, 1u, elected);
                        umma_pair_if<KIND>(d_tmem, a_lo + a_s3, a_hi, b_lo + b_s3, b_hi, idesc, 1u, elected);
                        umma_commit_pair_if(empty_bar(stage), pair_mask, elected);
                        if (kb == kb1 - 1) umma_commit_pair_if(tfull_bar(acc), pair_mask, elected);
                    }
                    accumulate = 1u;
                    __syncwarp();
                    soff += STAGE16;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; soff = 0; }
                }
                if (kb1 <= kb0) umma_commit_pair_if(tfull_bar(acc), pair_mask, elected);
            }
        }
    } else {
        // ------------------------------------------------ warps 2..9 (both CTAs, own 128 rows)
        // Warps 2-5: epilogue.  Warps 6-9: VNNI re-layout (if that is B's form), then the second half
        // of the epilogue in a pair that delivers a single tile (see the single-CTA kernel).
        const int set = warp >= 6 ? 1 : 0;
        const int quarter = warp & 3;
        uint8_t* staging = gen_base + STAGES * STAGE + quarter * 8192;
        if (set == 1 && B_VNNI) {
            // -------------------------------------------- VNNI re-layout
            // Each CTA re-lays its own HALF columns in place (see vnni_relayout_stage) and reports
            // each finished stage to the leader's full[] barrier.
            const int tw = warp - 6;
            const uint32_t lead_full0 = map_to_cta(full_bar(0), leader);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int unit = pair_id; ok && unit < total_units; unit += num_pairs) {
                int tile, split, gemm, kb0, kb1, tail;
                if (!decode(unit, tile, split, gemm, kb0, kb1, tail)) continue;
                for (int kb = kb0; kb < kb1; ++kb) {
                    // even stages: warps 6 and 7, odd stages: warps 8 and 9 (STAGES is even)
                    if ((stage & 1) == (tw >> 1)) {
                        if (!mbar_wait(raw_bar(stage), phase, abort_flag)) {
                            if (lane == 0) give_up(0x500u + stage);
                            ok = false;
                            break;
                        }
                        vnni_relayout_stage<HALF, 2>(smem_base + stage * STAGE + UMMA_A_STAGE_BYTES, tw & 1, lane);
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster_cta_release(lead_full0 + 8u * stage);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
        if (CLUSTER_REDUCE) {
            // -------------------------------------------- epilogue, K splits reduced inside the cluster
            // One unit per pair (grid = 2 x units); this pair's split = its index in the cluster.  The
            // other splits of this CTA's 128 rows are the CTAs with the same parity of cluster rank.
            int tile, split, gemm;
            umma_decode_unit(p, pair_id, tile, split, gemm);
            int mb, nb;
            umma_tile_coords(p, tile, mb, nb);
            bool ok = pair_id < total_units;
            const float* bias_sm = p.tma_store ? umma_park_bias<BN>(p, reinterpret_cast<float*>(staging + set * 2048), nb * BN, lane)
                                               : nullptr;
            if (ok && !mbar_wait(tfull_bar(0), 0u, abort_flag)) {
                if (lane == 0) give_up(0x400u);
                ok = false;
            }
            tc_fence_after_sync();
            umma_cluster_epilogue<BN>(p, &tmap_c, tmem_base, smem_base, gen_base, staging, bias_sm, quarter, set, lane,
                                      static_cast<uint32_t>(p.splits), crank >> 1, rank, 2u,
                                      mb * BM2 + static_cast<int>(rank) * UMMA_BM, nb * BN, gemm, ok, recv_bar0, abort_flag);
        } else if (set == 1) {
            // -------------------------------------------- second half of a one-shot epilogue
            if (one_shot && pair_id < total_units) {
                int tile, split, gemm, kb0, kb1, tail;
                if (!decode(pair_id, tile, split, gemm, kb0, kb1, tail)) tile = 0;
                int mb, nb;
                umma_tile_coords(p, tile, mb, nb);
                const float* bias_sm = umma_park_bias<BN>(p, reinterpret_cast<float*>(staging + 6144), nb * BN, lane);
                if (!mbar_wait(tfull_bar(0), 0u, abort_flag)) {
                    if (lane == 0) give_up(0x480u);
                } else {
                    tc_fence_after_sync();
                    umma_epilogue_oneshot<BN>(p, &tmap_c, tmem_base + (static_cast<uint32_t>(quarter * 32) << 16),
                                              gen_base + (quarter * 2 + 1) * (BN * 64),
                                              mb * BM2 + static_cast<int>(rank) * UMMA_BM + quarter * 32, nb * BN, gemm, lane,
                                              kb1 <= kb0, bias_sm, BN / 64, BN / 32);
                }
                if (lane == 0) bulk_wait_read<0>();
                __syncwarp();
            }
        } else {
            // -------------------------------------------- epilogue
            int local = 0;
            bool ok = true;
            for (int unit = pair_id; ok && unit < total_units; unit += num_pairs, ++local) {
                int tile, split, gemm, kb0, kb1, tail;
                if (!decode(unit, tile, split, gemm, kb0, kb1, tail)) continue;
                int mb, nb;
                umma_tile_coords(p, tile, mb, nb);
                const int acc = local & 1;
                const float* bias_smem = one_shot ? umma_park_bias<BN>(p, reinterpret_cast<float*>(staging + 4096), nb * BN, lane)
                                                  : umma_fetch_bias<BN>(p, staging, nb * BN, lane);
                if (!mbar_wait(tfull_bar(acc), (local >> 1) & 1u, abort_flag)) {
                    if (lane == 0) give_up(0x400u + acc);
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                const int row0 = mb * BM2 + static_cast<int>(rank) * UMMA_BM + quarter * 32;
                const bool empty_k = kb1 <= kb0;
                if (one_shot) {
                    // the only tile of this pair: the ring is idle, batch the stores through it (first half of
                    // the columns; warps 6-9 take the second)
                    umma_epilogue_oneshot<BN>(p, &tmap_c, tmem_base + acc * BN + (static_cast<uint32_t>(quarter * 32) << 16),
                                              gen_base + (quarter * 2) * (BN * 64), row0, nb * BN, gemm, lane, empty_k, bias_smem,
                                              0, BN / 64);
                    tc_fence_before_sync();
                    mbar_arrive_cluster_cta_release(map_to_cta(tempty_bar(acc), leader));
                    continue;
                }
                // FP32 partial of a K split: the [split][M][N] workspace, or this tail tile's own slab
                PartialDst pdst = {p.partial + (static_cast<size_t>(split) * p.gemms + gemm) * p.M * p.N, p.N, row0, 0, p.M, p.N};
                if (tail >= 0)
                    pdst = {p.partial + (static_cast<size_t>(tail) * p.sk_max_segs + split) * (BM2 * BN), BN,
                            static_cast<int>(rank) * UMMA_BM + quarter * 32, 0, BM2, BN};
                const PartialDst* pd = (p.splits > 1 || tail >= 0) ? &pdst : nullptr;
                const int pcol0 = tail >= 0 ? 0 : nb * BN;
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 64) {   // two 32-column chunks per round
                    uint32_t v0[32], v1[32];
                    const uint32_t taddr = tmem_base + acc * BN + c0 + (static_cast<uint32_t>(quarter * 32) << 16);
                    tmem_ld_32x32(taddr, v0);
                    tmem_ld_32x32(taddr + 32, v1);
                    tmem_ld_wait();
                    pdst.col0 = pcol0 + c0;
                    umma_store_chunk(p, &tmap_c, v0, row0, lane, nb * BN + c0, split, gemm, empty_k, staging, 0,
                                     bias_smem ? bias_smem + c0 : nullptr, pd);
                    __syncwarp();
                    pdst.col0 = pcol0 + c0 + 32;
                    umma_store_chunk(p, &tmap_c, v1, row0, lane, nb * BN + c0 + 32, split, gemm, empty_k, staging, 1,
                                     bias_smem ? bias_smem + c0 + 32 : nullptr, pd);
                    __syncwarp();
                }
                tc_fence_before_sync();
                mbar_arrive_cluster_cta_release(map_to_cta(tempty_bar(acc), leader));
            }
            if (lane == 0) bulk_wait_read<0>();   // this warp's TMA stores are done with the staging buffers
            __syncwarp();
        }
    }

    if (CLUSTER_REDUCE && warp < 2) {
        // the cluster barrier counts every thread: the other roles pass it here
        cluster_arrive();
        cluster_wait();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

}  // namespace nk
