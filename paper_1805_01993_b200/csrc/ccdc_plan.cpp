// Host planner: file placement (Section IV-A), function assignment
// (Section III, sets S_k) and the multicast schedule (Section IV-B) of the
// compressed CDC scheme, flattened into the offset tables the kernels walk.
// No CUDA call is made here.
#include <algorithm>
#include <climits>
#include <cstring>
#include <new>

#include "ccdc_internal.h"
#include "ccdc_stream.h"

namespace {

// C(n, k), or -1 when it does not fit 62 bits
long long choose(int n, int k) {
    if (k < 0 || k > n) return 0;
    k = std::min(k, n - k);
    unsigned __int128 c = 1;
    for (int i = 1; i <= k; ++i) {
        c = c * (unsigned)(n - k + i) / (unsigned)i;
        if (c > ((unsigned __int128)1 << 62)) return -1;
    }
    return (long long)c;
}

// lexicographic rank of the ascending m-subset c of {0..n-1}: the number of
// m-subsets that precede it = those that agree on the first i entries and
// carry a smaller value v at position i
long long subset_rank(const int *c, int m, int n) {
    long long rank = 0;
    int lo = 0;
    for (int i = 0; i < m; ++i) {
        for (int v = lo; v < c[i]; ++v) rank += choose(n - 1 - v, m - 1 - i);
        lo = c[i] + 1;
    }
    return rank;
}

// inverse of subset_rank
void subset_unrank(long long rank, int m, int n, int *c) {
    int v = 0;
    for (int i = 0; i < m; ++i) {
        for (;; ++v) {
            long long cnt = choose(n - 1 - v, m - 1 - i);
            if (rank < cnt) break;
            rank -= cnt;
        }
        c[i] = v++;
    }
}

int index_in(const int *set, int m, int x) {
    for (int i = 0; i < m; ++i) if (set[i] == x) return i;
    return -1;
}

long long seg_valid(const ccdc_plan_s &P, int i) {
    long long rest = P.len - (long long)i * P.s;
    return std::max(0LL, std::min(P.s, rest));
}

// operand reference; a segment that does not exist (vl = 0) is never
// dereferenced and gets offset 0 so that every stored offset is in bounds
ccdc_ref seg_ref(long long off, long long vl) { return vl > 0 ? ccdc_ref{off, vl} : ccdc_ref{0, 0}; }

// first element of the packet row (batch p, first file, functions of node t) in node k's partition
long long part_row(const ccdc_plan_s &P, int k, long long p, int t) {
    return P.slot[(size_t)k * P.nbatch + p] * P.b * P.row_elems + (long long)t * P.len;
}

// index of packet (batch p, for node t) among node k's packets: [local batch][outside node ascending]
long long packet_index(const ccdc_plan_s &P, int k, long long p, int t) {
    const int *lab = &P.batch_nodes[(size_t)p * P.r];
    int before = 0;                          // members of the label smaller than t
    for (int i = 0; i < P.r; ++i) if (lab[i] < t) ++before;
    return P.slot[(size_t)k * P.nbatch + p] * (P.K - P.r) + (t - before);
}

int check_parameters(int K, int r, long long N, int Q, long long B, int dtype) {
    if (K < 2 || K > CCDC_MAX_K) return CCDC_EINVAL;
    if (r < 1 || r > K - 1) return CCDC_EINVAL;            // mu*K in {1..K-1}
    if (N < K) return CCDC_EINVAL;                         // K <= N
    if (Q < K || Q % K != 0) return CCDC_EINVAL;           // K | Q
    if (B < 1) return CCDC_EINVAL;
    if (dtype != CCDC_I32 && dtype != CCDC_F32) return CCDC_EINVAL;
    if (N > (1LL << 40) || B > (1LL << 40) || Q > (1 << 24)) return CCDC_ESIZE;
    return CCDC_OK;
}

// Launch shape of the fused decode over `nout` output rows: block size, files
// of a batch whose loads are issued together, and the split of the batch loop
// over blocks.  P.sm_count is 148 (B200) until the tables are uploaded, when
// the device's own count replaces it.
long long decode_tiles_per_seg(const ccdc_plan_s &P, int threads) {
    // the bulk-copy pipeline covers a fixed number of words per block, whatever the vector width
    const long long tile = P.family == 1 ? CCDC_STREAM_TILE_WORDS : (long long)threads * P.vec * CCDC_DECODE_VECTORS;
    return (P.s + tile - 1) / tile;
}

void set_split(ccdc_plan_s &P, long long nchunk) {
    nchunk = std::max(1LL, std::min(nchunk, P.nterm));
    P.terms_per_chunk = (P.nterm + nchunk - 1) / nchunk;
    P.nchunk = (int)((P.nterm + P.terms_per_chunk - 1) / P.terms_per_chunk);
    // up to 8 chunks (the portable cluster size) of the kernel form that loads several files together:
    // the partial sums meet in a thread-block cluster, no workspace
    P.decode_cluster = CCDC_DECODE_CLUSTER_SUM && P.family == 0 && P.decode_files > 1 && P.nchunk >= 2 && P.nchunk <= 8 &&
                       P.device_has_bulk_copies;
}

void choose_split(ccdc_plan_s &P, long long nout) {
    // files of a batch loaded together: all of a small batch, fewer while a batch
    // (coded word + r-1 operands) would keep more than 40 words per thread in flight
    int group = P.b <= 1 ? 1 : P.b == 2 ? 2 : 4;
    group = std::min(group, CCDC_DECODE_FILES_MAX);
    while (group > 1 && (1 + (P.r - 1) * group) * P.vec > CCDC_DECODE_GROUP_WORDS) group /= 2;
    if (P.r > 4 || P.vec < 2) group = 1;
    // 0: the batch-by-batch kernel (any r, any number of files); 1: one-file batches
    P.decode_files = (P.r > 4 || P.vec < 2 || (group == 1 && P.b > 1)) ? 0 : group;
    // several files per batch: many registers per thread, so small blocks
    P.decode_threads = group > 1 ? CCDC_DECODE_THREADS_FILES : CCDC_DECODE_THREADS;
    // blocks resident per SM at the registers these kernels take
    auto resident = [&](int threads) {
        if (P.family == 1) return (long long)P.sm_count * 3;       // bulk-copy pipeline: shared memory for three blocks
        if (threads == CCDC_DECODE_THREADS_FILES && group > 1) return (long long)P.sm_count * CCDC_DECODE_BLOCKS_FILES(P.vec);
        return (long long)P.sm_count * (threads >= 1024 ? 1 : threads >= 512 ? 3 : 768 / threads);
    };
    // enough thread blocks to fill the GPU (8 per SM) while a block still walks a fair number of batches
    auto many_blocks = [&](int threads) {
        const long long base = std::max(1LL, nout * P.r * decode_tiles_per_seg(P, threads));
        const long long want = ((long long)P.sm_count * 8 + base - 1) / base;
        return std::max(1LL, std::min(want, std::max(1LL, P.nterm / 8)));
    };
    set_split(P, many_blocks(P.decode_threads));
    const long long base = std::max(1LL, nout * P.r * decode_tiles_per_seg(P, P.decode_threads));
    if (base * P.nchunk < 6 * resident(P.decode_threads)) {
        // A launch of a few waves only: the rounding of the last wave decides.  Take the split with
        // the fewest (waves x batches per block), a block costing two batches' time to start and end.
        long long best = 0, best_cost = 0;
        for (long long n = 1; n <= std::max(1LL, P.nterm / 4); ++n) {
            const long long per = (P.nterm + n - 1) / n, real = (P.nterm + per - 1) / per;
            if (real != n) continue;
            const long long waves = (base * n + resident(P.decode_threads) - 1) / resident(P.decode_threads);
            if (waves > 6) break;
            const long long cost = waves * (per + 2);
            if (best == 0 || cost < best_cost) { best = n; best_cost = cost; }
        }
        if (best) set_split(P, best);
    }
    // short segments of one-file batches: one large block per segment instead of two smaller ones, but only
    // when the launch still has many waves of them (one such block is resident per SM); measured: K=16, r=4
    // gains 0.6 %, K=10, r=3 with 450 blocks would lose 17 %
    if (P.family == 0 && group <= 1 && P.s <= (long long)CCDC_DECODE_THREADS_SHORT * P.vec * CCDC_DECODE_VECTORS &&
        P.s > (long long)CCDC_DECODE_THREADS * P.vec * CCDC_DECODE_VECTORS) {
        const long long n = many_blocks(CCDC_DECODE_THREADS_SHORT);
        const long long per = (P.nterm + n - 1) / n, real = (P.nterm + per - 1) / per;
        const long long blocks = nout * P.r * decode_tiles_per_seg(P, CCDC_DECODE_THREADS_SHORT) * real;
        if (blocks >= (long long)P.sm_count * 6) {
            P.decode_threads = CCDC_DECODE_THREADS_SHORT;
            set_split(P, n);
        }
    }
}

// Restrict a finished plan to the nodes of one rank out of `world` (node k lives
// on rank k / (K/world)).  The rank encodes the coded rows its nodes send, into a
// send buffer of its own; after an all-gather of the send buffers (rank-major)
// coded row (round, a) sits at coded_row_pos; the rank decodes for its nodes.
int apply_shard(ccdc_plan_s &P, int rank, int world) {
    const int K = P.K, r = P.r;
    if (world < 1 || rank < 0 || rank >= world || K % world != 0) return CCDC_EINVAL;
    const int per = K / world;
    const long long nrows = P.nround * (r + 1);
    P.shard_rank = rank; P.shard_world = world;
    P.coded_row_pos.assign(nrows, 0);
    std::vector<long long> count(world, 0);
    for (long long cr = 0; cr < nrows; ++cr) {
        const int owner = P.round_group[cr] / per;          // round_group is [round][a] = sender of row cr
        P.coded_row_pos[cr] = count[owner]++;
    }
    for (int w = 1; w < world; ++w) if (count[w] != count[0]) return CCDC_EINVAL;
    P.send_rows = count[0];
    for (long long cr = 0; cr < nrows; ++cr) P.coded_row_pos[cr] += (P.round_group[cr] / per) * P.send_rows;
    // encode: only the rows this rank's nodes send, packed into its send buffer
    ccdc_gather_table enc;
    enc.na = P.enc_fused.na; enc.n_max = P.enc_fused.n_max;
    for (long long cr = 0; cr < nrows; ++cr) {
        if (P.round_group[cr] / per != rank) continue;
        ccdc_row R = P.enc_fused.rows[cr];
        R.dst_off = (P.coded_row_pos[cr] - rank * P.send_rows) * P.s_pad;
        enc.rows.push_back(R);
        for (int a = 0; a < enc.na; ++a) enc.refs.push_back(P.enc_fused.refs[(size_t)cr * enc.na + a]);
    }
    P.enc_fused = enc;
    // decode: coded rows are found at their gathered positions
    for (size_t x = 0; x < P.dec_terms.size(); x += P.term_stride) {
        ccdc_ref &c = P.dec_terms[x];
        if (c.off >= 0) c.off = P.coded_row_pos[c.off / P.s_pad] * P.s_pad;
    }
    P.out_rows.clear();
    for (long long j = 0; j < P.J; ++j)
        for (int k = rank * per; k < (rank + 1) * per; ++k) P.out_rows.push_back((int)(j * K + k));
    choose_split(P, (long long)P.out_rows.size());
    return CCDC_OK;
}

// everything that follows from batches + rounds
int finish(ccdc_plan_s &P) {
    const int K = P.K, r = P.r;
    // storage
    P.slot.assign((size_t)K * P.nbatch, -1);
    P.nlocal.assign(K, 0);
    for (long long p = 0; p < P.nbatch; ++p)
        for (int i = 0; i < r; ++i) {
            int k = P.batch_nodes[(size_t)p * r + i];
            P.slot[(size_t)k * P.nbatch + p] = P.nlocal[k]++;
        }
    P.node_nfiles.assign(K, 0);
    for (int k = 0; k < K; ++k) P.node_nfiles[k] = P.nlocal[k] * P.b;
    // who receives which batch in which round; every (batch, outside node) exactly once
    P.recv_round.assign((size_t)P.nbatch * K, -1);
    P.node_round_index.assign((size_t)P.nround * (r + 1), 0);
    P.node_nrounds.assign(K, 0);
    for (long long g = 0; g < P.nround; ++g) {
        const int *S = &P.round_group[(size_t)g * (r + 1)];
        for (int a = 0; a <= r; ++a) {
            long long p = P.round_batch[(size_t)g * (r + 1) + a];
            if (p < 0 || p >= P.nbatch) return CCDC_EINVAL;
            const int *lab = &P.batch_nodes[(size_t)p * r];
            for (int x = 0, y = 0; x <= r; ++x) {          // label must be S without S[a]
                if (x == a) continue;
                if (lab[y++] != S[x]) return CCDC_EINVAL;
            }
            long long &slot = P.recv_round[(size_t)p * K + S[a]];
            if (slot != -1) return CCDC_EINVAL;
            slot = g;
            P.node_round_index[(size_t)g * (r + 1) + a] = P.node_nrounds[S[a]]++;
        }
    }
    for (long long p = 0; p < P.nbatch; ++p)
        for (int k = 0; k < K; ++k) {
            bool inside = index_in(&P.batch_nodes[(size_t)p * r], r, k) >= 0;
            if (inside != (P.recv_round[(size_t)p * K + k] == -1)) return CCDC_EINVAL;
        }

    // vector width: every segment start and length must be a multiple of it
    P.vec = (P.s % 4 == 0 && P.len % 4 == 0) ? 4 : (P.s % 2 == 0 && P.len % 2 == 0) ? 2 : 1;
    P.term_stride = 1 + std::max(r - 1, 1);

    const long long nrows = P.nround * (r + 1);
    // ---- fused encode: coded row <- r partition segments of the sender
    // ---- stepwise encode: the same from the sender's materialised packets
    P.enc_fused.na = P.enc_pk.na = r;
    P.enc_fused.n_max = P.enc_pk.n_max = P.s;
    P.enc_fused.rows.resize(nrows); P.enc_fused.refs.resize((size_t)nrows * r);
    P.enc_pk.rows.resize(nrows);    P.enc_pk.refs.resize((size_t)nrows * r);
    for (long long g = 0; g < P.nround; ++g) {
        const int *S = &P.round_group[(size_t)g * (r + 1)];
        const long long *bat = &P.round_batch[(size_t)g * (r + 1)];
        for (int as = 0; as <= r; ++as) {
            const long long cr = g * (r + 1) + as;
            const int ks = S[as];
            ccdc_row row{ks, 0, cr * P.s_pad, P.s, -1, 0};
            P.enc_fused.rows[cr] = row;
            P.enc_pk.rows[cr] = row;
            int n = 0;
            for (int a = 0; a <= r; ++a) {
                if (a == as) continue;
                const long long p = bat[a];
                const int i = index_in(&P.batch_nodes[(size_t)p * r], r, ks);
                const long long vl = seg_valid(P, i);
                P.enc_fused.refs[(size_t)cr * r + n] = seg_ref(part_row(P, ks, p, S[a]) + (long long)i * P.s, vl);
                P.enc_pk.refs[(size_t)cr * r + n] = seg_ref(packet_index(P, ks, p, S[a]) * P.len + (long long)i * P.s, vl);
                ++n;
            }
        }
    }
    // ---- stepwise combine: packet <- sum over the batch's files
    P.cmb.na = 1; P.cmb.n_max = P.len;
    for (int k = 0; k < K; ++k)
        for (long long p = 0; p < P.nbatch; ++p) {
            if (P.slot[(size_t)k * P.nbatch + p] < 0) continue;
            for (int t = 0; t < K; ++t) {
                if (index_in(&P.batch_nodes[(size_t)p * r], r, t) >= 0) continue;
                P.cmb.rows.push_back({k, k, packet_index(P, k, p, t) * P.len, P.len, -1, 0});
                P.cmb.refs.push_back({part_row(P, k, p, t), P.len});
            }
        }
    // ---- stepwise decode: decoded segment <- coded XOR r-1 own packet segments
    const int r1 = r - 1;
    P.dec_pk.na = r1; P.dec_pk.n_max = P.s;
    for (long long g = 0; g < P.nround; ++g) {
        const int *S = &P.round_group[(size_t)g * (r + 1)];
        const long long *bat = &P.round_batch[(size_t)g * (r + 1)];
        for (int ak = 0; ak <= r; ++ak) {
            const int k = S[ak];
            const long long ridx = P.node_round_index[(size_t)g * (r + 1) + ak];
            for (int as = 0; as <= r; ++as) {
                if (as == ak) continue;
                const int ks = S[as];
                const int i0 = index_in(&P.batch_nodes[(size_t)bat[ak] * r], r, ks);
                const long long n0 = seg_valid(P, i0);
                P.dec_pk.rows.push_back({k, k, n0 > 0 ? ridx * P.len + (long long)i0 * P.s : 0, n0,
                                         (g * (r + 1) + as) * P.s_pad, 0});
                for (int a = 0; a <= r; ++a) {
                    if (a == ak || a == as) continue;
                    const int i = index_in(&P.batch_nodes[(size_t)bat[a] * r], r, ks);
                    P.dec_pk.refs.push_back(seg_ref(packet_index(P, k, bat[a], S[a]) * P.len + (long long)i * P.s,
                                                    seg_valid(P, i)));
                }
            }
        }
    }
    // ---- fused decode + reduce, and the stepwise reduce
    const int TS = P.term_stride;
    const long long nout = P.J * K;
    P.dec_terms.assign((size_t)nout * r * P.nterm * TS, ccdc_ref{-1, 0});
    P.red_terms.resize((size_t)nout * P.nterm);
    for (long long j = 0; j < P.J; ++j)
        for (int k = 0; k < K; ++k) {
            const long long orow = j * K + k;
            for (long long tt = 0; tt < P.nterm; ++tt) {
                const long long p = P.job_batch0[j] + tt;
                if (P.batch_job[p] != j) return CCDC_EINVAL;
                const bool local = P.slot[(size_t)k * P.nbatch + p] >= 0;
                const long long g = local ? -1 : P.recv_round[(size_t)p * K + k];
                P.red_terms[(size_t)orow * P.nterm + tt] = local
                    ? ccdc_ref{part_row(P, k, p, k), 0}
                    : ccdc_ref{P.node_round_index[(size_t)g * (r + 1) +
                                   index_in(&P.round_group[(size_t)g * (r + 1)], r + 1, k)] * P.len, 1};
                for (int i = 0; i < r; ++i) {
                    ccdc_ref *e = &P.dec_terms[(((size_t)orow * r + i) * P.nterm + tt) * TS];
                    if (local) {
                        e[0] = {-1, 0};
                        e[1] = seg_ref(part_row(P, k, p, k) + (long long)i * P.s, seg_valid(P, i));
                        continue;
                    }
                    const int *S = &P.round_group[(size_t)g * (r + 1)];
                    const long long *bat = &P.round_batch[(size_t)g * (r + 1)];
                    const int ak = index_in(S, r + 1, k);
                    const int ks = P.batch_nodes[(size_t)p * r + i];    // sender whose label is segment i
                    const int as = index_in(S, r + 1, ks);
                    e[0] = {(g * (r + 1) + as) * P.s_pad, P.s};
                    int n = 1;
                    for (int a = 0; a <= r; ++a) {
                        if (a == ak || a == as) continue;
                        const int i2 = index_in(&P.batch_nodes[(size_t)bat[a] * r], r, ks);
                        e[n++] = seg_ref(part_row(P, k, bat[a], S[a]) + (long long)i2 * P.s, seg_valid(P, i2));
                    }
                }
            }
        }

    choose_split(P, nout);

    // ---- every offset must stay inside its buffer
    auto check_table = [&](const ccdc_gather_table &T, bool src_is_packets, bool dst_kind_coded,
                           bool dst_is_packets, long long nf) -> bool {
        for (size_t x = 0; x < T.rows.size(); ++x) {
            const ccdc_row &R = T.rows[x];
            if (R.src_node < 0 || R.src_node >= K || R.n < 0 || R.dst_off < 0) return false;
            long long dst_cap = dst_kind_coded ? nrows * P.s_pad
                              : dst_is_packets ? P.nlocal[R.dst_node] * (K - r) * P.len
                                               : P.node_nrounds[R.dst_node] * P.len;
            if (R.dst_off + R.n > dst_cap) return false;
            if (R.coded_off >= 0 && R.coded_off + R.n > nrows * P.s_pad) return false;
            long long src_cap = src_is_packets ? P.nlocal[R.src_node] * (K - r) * P.len
                                               : P.nlocal[R.src_node] * P.b * P.row_elems;
            for (int a = 0; a < T.na; ++a) {
                const ccdc_ref &E = T.refs[x * T.na + a];
                if (E.off < 0 || E.vl < 0 || E.vl > T.n_max) return false;
                long long last = E.off + (nf - 1) * P.row_elems + std::min(E.vl, R.n);
                if (last > src_cap) return false;
            }
        }
        return true;
    };
    if (!check_table(P.enc_fused, false, true, false, P.b)) return CCDC_EINVAL;
    if (!check_table(P.enc_pk, true, true, false, 1)) return CCDC_EINVAL;
    if (!check_table(P.cmb, false, false, true, P.b)) return CCDC_EINVAL;
    if (!check_table(P.dec_pk, true, false, false, 1)) return CCDC_EINVAL;
    for (long long orow = 0; orow < nout; ++orow) {
        const int k = (int)(orow % K);
        const long long cap = P.nlocal[k] * P.b * P.row_elems;
        for (size_t x = 0; x < (size_t)r * P.nterm; ++x) {
            const ccdc_ref *e = &P.dec_terms[((size_t)orow * r * P.nterm + x) * TS];
            const int nref = e[0].off < 0 ? 1 : r1;
            if (e[0].off >= 0 && e[0].off + P.s > nrows * P.s_pad) return CCDC_EINVAL;
            for (int c = 1; c <= nref; ++c)
                if (e[c].off < 0 || e[c].off + (P.b - 1) * P.row_elems + e[c].vl > cap) return CCDC_EINVAL;
        }
    }
    return CCDC_OK;
}

int make_plan(int K, int r, long long N, int Q, long long B, ccdc_dtype_t dtype, bool jobs, ccdc_plan_t **out,
              int gamma = 1) {
    if (!out) return CCDC_EINVAL;
    *out = nullptr;
    int rc = check_parameters(K, r, N, Q, B, (int)dtype);
    if (rc != CCDC_OK) return rc;
    const long long n_rsub = choose(K, r), n_r1sub = choose(K, r + 1);
    if (n_rsub <= 0 || n_r1sub <= 0 || n_r1sub > (1LL << 24)) return CCDC_ESIZE;
    {   // the decode's term table alone: out rows x r segments x batches per job x refs of 16 bytes
        const long double jobs_n = jobs ? (long double)gamma * n_r1sub : 1.0L;
        const long double terms = jobs_n * K * r * (jobs ? r + 1 : n_rsub) * (1 + std::max(r - 1, 1)) * 16.0L;
        if (terms > 2.0e9L) return CCDC_ESIZE;              // host and device tables of more than 2 GB
    }
    if (!jobs && N % n_rsub != 0) return CCDC_EINVAL;       // batches of equal size
    if (jobs && N % (r + 1) != 0) return CCDC_EINVAL;
    if (gamma < 1 || (!jobs && gamma != 1)) return CCDC_EINVAL;
    if ((long long)gamma * n_r1sub > (1LL << 24)) return CCDC_ESIZE;
    try {
        ccdc_plan_s *pp = new ccdc_plan_s();
        ccdc_plan_s &P = *pp;
        P.K = K; P.r = r; P.N = N; P.Q = Q; P.B = B; P.dtype = (int)dtype; P.jobs_mode = jobs;
        P.len = (long long)(Q / K) * B;
        P.s = (P.len + r - 1) / r;
        P.s_pad = (P.s + 3) / 4 * 4;
        P.row_elems = (long long)Q * B;
        int c[CCDC_MAX_K + 1], rest[CCDC_MAX_K + 1];
        if (!jobs) {
            P.J = 1; P.b = N / n_rsub; P.nbatch = n_rsub; P.nround = n_r1sub; P.nterm = n_rsub;
            P.job_batch0.assign(1, 0);
            P.batch_nodes.resize((size_t)P.nbatch * r);
            P.batch_file0.resize(P.nbatch); P.batch_job.assign(P.nbatch, 0);
            for (long long p = 0; p < P.nbatch; ++p) {
                subset_unrank(p, r, K, &P.batch_nodes[(size_t)p * r]);
                P.batch_file0[p] = p * P.b;
            }
            P.round_group.resize((size_t)P.nround * (r + 1));
            P.round_batch.resize((size_t)P.nround * (r + 1));
            for (long long g = 0; g < P.nround; ++g) {
                subset_unrank(g, r + 1, K, c);
                std::memcpy(&P.round_group[(size_t)g * (r + 1)], c, sizeof(int) * (r + 1));
                for (int a = 0; a <= r; ++a) {
                    for (int x = 0, y = 0; x <= r; ++x) if (x != a) rest[y++] = c[x];
                    P.round_batch[(size_t)g * (r + 1) + a] = subset_rank(rest, r, K);
                }
            }
        } else {
            // gamma groups of C(K, r+1) jobs: job j lives on subset j mod C(K, r+1); the groups are
            // independent repetitions of the same operations (Section IV: J = gamma * C(K, mu K + 1))
            P.J = (long long)gamma * n_r1sub; P.b = N / (r + 1); P.nbatch = P.J * (r + 1); P.nround = P.J * (K - r);
            P.nterm = r + 1;
            P.job_batch0.resize(P.J);
            P.batch_nodes.resize((size_t)P.nbatch * r);
            P.batch_file0.resize(P.nbatch); P.batch_job.resize(P.nbatch);
            // the a-th size-r subset of an (r+1)-set in lexicographic order
            // omits its (r-a)-th member
            for (long long j = 0; j < P.J; ++j) {
                subset_unrank(j % n_r1sub, r + 1, K, c);
                P.job_batch0[j] = j * (r + 1);
                for (int a = 0; a <= r; ++a) {
                    const long long p = j * (r + 1) + a;
                    for (int x = 0, y = 0; x <= r; ++x) if (x != r - a) P.batch_nodes[(size_t)p * r + y++] = c[x];
                    P.batch_job[p] = j;
                    P.batch_file0[p] = j * N + a * P.b;
                }
            }
            P.round_group.resize((size_t)P.nround * (r + 1));
            P.round_batch.resize((size_t)P.nround * (r + 1));
            long long g = 0;
            for (long long j = 0; j < P.J; ++j) {
                subset_unrank(j % n_r1sub, r + 1, K, c);
                const long long group0 = j / n_r1sub * n_r1sub;     // first job of j's group
                // stage 1: member a receives job j's batch that omits it
                std::memcpy(&P.round_group[(size_t)g * (r + 1)], c, sizeof(int) * (r + 1));
                for (int a = 0; a <= r; ++a) P.round_batch[(size_t)g * (r + 1) + a] = j * (r + 1) + (r - a);
                ++g;
                // stage 2: one round per outside node i
                for (int i = 0; i < K; ++i) {
                    if (index_in(c, r + 1, i) >= 0) continue;
                    std::memcpy(&P.round_group[(size_t)g * (r + 1)], c, sizeof(int) * (r + 1));
                    for (int a = 0; a <= r; ++a) {
                        // home of the job = {i} U S\{S[a]}, ascending; m = position of i in it
                        int m = 0, y = 0;
                        bool placed = false;
                        for (int x = 0; x <= r; ++x) {
                            if (x == a) continue;
                            if (!placed && i < c[x]) { m = y; rest[y++] = i; placed = true; }
                            rest[y++] = c[x];
                        }
                        if (!placed) { m = y; rest[y++] = i; }
                        const long long jt = group0 + subset_rank(rest, r + 1, K);
                        P.round_batch[(size_t)g * (r + 1) + a] = jt * (r + 1) + (r - m);
                    }
                    ++g;
                }
            }
            if (g != P.nround) { delete pp; return CCDC_EINVAL; }
        }
        rc = finish(P);
        if (rc != CCDC_OK) { delete pp; return rc; }
        *out = pp;
        return CCDC_OK;
    } catch (const std::bad_alloc &) {
        return CCDC_ENOMEM;
    }
}

// The appendix's compression-only scheme for one job, mu = r/K: m = ceil(K/r)
// batches (the first m-1 of mu*N files, the last the rest), node k stores batch
// k mod m, and for every batch t it lacks node k is sent one pre-combined packet
// by the first node after k (cyclically) that stores batch t.
int make_compression_plan(int K, int r, long long N, int Q, long long B, ccdc_dtype_t dtype, ccdc_plan_t **out) {
    if (!out) return CCDC_EINVAL;
    *out = nullptr;
    int rc = check_parameters(K, r, N, Q, B, (int)dtype);
    if (rc != CCDC_OK) return rc;
    if (((long long)r * N) % K != 0) return CCDC_EINVAL;        // mu*N files per batch
    const int m = (K + r - 1) / r;
    const long long full = (long long)r * N / K, last = N - (long long)(m - 1) * full;
    if (last < 1) return CCDC_EINVAL;
    try {
        ccdc_plan_s *pp = new ccdc_plan_s();
        ccdc_plan_s &P = *pp;
        P.K = K; P.r = r; P.N = N; P.Q = Q; P.B = B; P.dtype = (int)dtype; P.compression_mode = true;
        P.J = 1; P.b = full; P.len = (long long)(Q / K) * B; P.s = P.len; P.s_pad = (P.s + 3) / 4 * 4;
        P.row_elems = (long long)Q * B;
        P.nbatch = m; P.nround = 0; P.nterm = m;
        P.vec = P.len % 4 == 0 ? 4 : P.len % 2 == 0 ? 2 : 1;
        P.term_stride = 2;
        P.job_batch0.assign(1, 0);
        P.batch_file0.resize(m); P.batch_job.assign(m, 0);
        for (int t = 0; t < m; ++t) P.batch_file0[t] = t * full;
        P.slot.assign((size_t)K * m, -1);
        P.nlocal.assign(K, 1); P.node_nfiles.assign(K, 0); P.node_nrounds.assign(K, m - 1);
        for (int k = 0; k < K; ++k) {
            P.slot[(size_t)k * m + k % m] = 0;
            P.node_nfiles[k] = (k % m == m - 1) ? last : full;
        }
        P.cmb.na = 1; P.cmb.n_max = P.len; P.cmb.uniform = false; P.cmb.nf_max = std::max(full, last);
        P.red_terms.resize((size_t)K * m);
        for (int k = 0; k < K; ++k) {
            int slot = 0;
            for (int t = 0; t < m; ++t) {
                const long long nf = t == m - 1 ? last : full;
                if (t == k % m) {
                    P.red_terms[(size_t)k * m + t] = {(long long)k * P.len, -nf};    // own batch, nf files
                    continue;
                }
                int ks = (k + 1) % K;
                while (ks % m != t) ks = (ks + 1) % K;
                P.cmb.rows.push_back({ks, k, (long long)slot * P.len, P.len, -1, nf});
                P.cmb.refs.push_back({(long long)k * P.len, P.len});
                P.red_terms[(size_t)k * m + t] = {(long long)slot * P.len, 1};
                ++slot;
            }
        }
        *out = pp;
        return CCDC_OK;
    } catch (const std::bad_alloc &) {
        return CCDC_ENOMEM;
    }
}

}  // namespace

void ccdc_internal_build_stream_tables(ccdc_plan_s *plan) {
    ccdc_plan_s &P = *plan;
    const int r = P.r, r1 = r - 1, TS = P.term_stride;
    const long long nb = P.b;
    // ---- decode: per output segment (out row, segment i) the rows of every batch, ascending
    ccdc_stream_table &D = P.dec_stream;
    D.rows.clear(); D.cells.clear(); D.chunk_row0.clear();
    const long long nout = P.J * P.K;
    for (long long orow = 0; orow < nout; ++orow)
        for (int i = 0; i < r; ++i) {
            const int seglen = (int)seg_valid(P, i);
            ccdc_stream_cell C = {(long long)D.rows.size(), orow * P.len + (long long)i * P.s, (int)(orow % P.K), seglen};
            for (long long tt = 0; tt < P.nterm; ++tt) {
                if (tt % P.terms_per_chunk == 0) D.chunk_row0.push_back((int)((long long)D.rows.size() - C.row0));
                const ccdc_ref *e = &P.dec_terms[(((size_t)orow * r + i) * P.nterm + tt) * TS];
                if (e[0].off < 0) {                         // a batch stored at the node: its files
                    for (long long f = 0; f < nb; ++f)
                        D.rows.push_back({e[1].off + f * P.row_elems, seglen,
                                          CCDC_SROW_FIRST_OP | CCDC_SROW_LAST_OP | (f == 0 ? CCDC_SROW_FIRST_FILE : 0) |
                                              (f == nb - 1 ? CCDC_SROW_LAST_FILE : 0)});
                    continue;
                }
                D.rows.push_back({e[0].off, seglen,
                                  CCDC_SROW_FROM_CODED | CCDC_SROW_CODED | CCDC_SROW_FIRST_OP | CCDC_SROW_FIRST_FILE |
                                      CCDC_SROW_LAST_FILE | (r1 == 0 ? CCDC_SROW_LAST_OP : 0)});
                for (int c = 1; c <= r1; ++c)
                    for (long long f = 0; f < nb; ++f)
                        D.rows.push_back({e[c].vl > 0 ? e[c].off + f * P.row_elems : 0, (int)std::min<long long>(seglen, e[c].vl),
                                          (c == r1 ? CCDC_SROW_LAST_OP : 0) | (f == 0 ? CCDC_SROW_FIRST_FILE : 0) |
                                              (f == nb - 1 ? CCDC_SROW_LAST_FILE : 0)});
            }
            D.chunk_row0.push_back((int)((long long)D.rows.size() - C.row0));
            D.cells.push_back(C);
        }
    // ---- encode: per coded row the files of its r operands
    ccdc_stream_table &E = P.enc_stream;
    E.rows.clear(); E.cells.clear(); E.chunk_row0.clear();
    const ccdc_gather_table &T = P.enc_fused;
    for (size_t x = 0; x < T.rows.size(); ++x) {
        const ccdc_row &R = T.rows[x];
        E.cells.push_back({(long long)E.rows.size(), R.dst_off, R.src_node, (int)R.n});
        E.chunk_row0.push_back(0);
        for (int a = 0; a < r; ++a) {
            const ccdc_ref &ref = T.refs[x * r + a];
            for (long long f = 0; f < nb; ++f)
                E.rows.push_back({ref.vl > 0 ? ref.off + f * P.row_elems : 0, (int)std::min(R.n, ref.vl),
                                  (a == 0 ? CCDC_SROW_FIRST_OP : 0) | (a == r - 1 ? CCDC_SROW_LAST_OP : 0) |
                                      (f == 0 ? CCDC_SROW_FIRST_FILE : 0) | (f == nb - 1 ? CCDC_SROW_LAST_FILE : 0)});
        }
        E.chunk_row0.push_back((int)(r * nb));
    }
}

void ccdc_internal_choose_split(ccdc_plan_s *plan) {
    if (plan->compression_mode || plan->tuned) return;
    choose_split(*plan, plan->shard_world > 1 ? (long long)plan->out_rows.size() : plan->J * plan->K);
}

void ccdc_internal_resplit(ccdc_plan_s *plan, int sm_count) {
    if (sm_count < 1 || sm_count == plan->sm_count) return;
    plan->sm_count = sm_count;
    if (plan->compression_mode || plan->tuned) return;
    choose_split(*plan, plan->shard_world > 1 ? (long long)plan->out_rows.size() : plan->J * plan->K);
}

extern "C" {

int ccdc_plan_sharded(int K, int r, long long N, int Q, long long B, ccdc_dtype_t dtype, int jobs, int rank,
                      int world, ccdc_plan_t **out) {
    int rc = make_plan(K, r, N, Q, B, dtype, jobs != 0, out);
    if (rc != CCDC_OK) return rc;
    rc = apply_shard(**out, rank, world);
    if (rc != CCDC_OK) { delete *out; *out = nullptr; }
    return rc;
}

long long ccdc_plan_coded_row_position(const ccdc_plan_t *p, long long g, int a) {
    if (!p || g < 0 || g >= p->nround || a < 0 || a > p->r) return -1;
    const long long cr = g * (p->r + 1) + a;
    return p->shard_world > 1 ? p->coded_row_pos[cr] : cr;
}

size_t ccdc_coded_send_bytes(const ccdc_plan_t *p) {
    if (!p) return 0;
    const long long rows = p->shard_world > 1 ? p->send_rows : p->nround * (p->r + 1);
    return (size_t)(rows * p->s_pad) * 4;
}

int ccdc_plan_node_is_local(const ccdc_plan_t *p, int k) {
    if (!p || k < 0 || k >= p->K) return 0;
    return k / (p->K / p->shard_world) == p->shard_rank;
}

int ccdc_plan_compression(int K, int r, long long N, int Q, long long B, ccdc_dtype_t dtype, ccdc_plan_t **out) {
    return make_compression_plan(K, r, N, Q, B, dtype, out);
}

long long ccdc_plan_batch_files(const ccdc_plan_t *p, long long b) {
    if (!p || b < 0 || b >= p->nbatch) return 0;
    if (p->compression_mode && b == p->nbatch - 1) return p->N - (p->nbatch - 1) * p->b;
    return p->b;
}

int ccdc_plan(int K, int r, long long N, int Q, long long B, ccdc_dtype_t dtype, ccdc_plan_t **out) {
    return make_plan(K, r, N, Q, B, dtype, false, out);
}

int ccdc_plan_jobs(int K, int r, long long N, int Q, long long B, ccdc_dtype_t dtype, ccdc_plan_t **out) {
    return make_plan(K, r, N, Q, B, dtype, true, out);
}

int ccdc_plan_jobs_gamma(int K, int r, long long N, int Q, long long B, ccdc_dtype_t dtype, int gamma,
                         ccdc_plan_t **out) {
    return make_plan(K, r, N, Q, B, dtype, true, out, gamma);
}

void ccdc_plan_destroy(ccdc_plan_t *plan) {
    if (!plan) return;
    ccdc_internal_release_device(plan);
    delete plan;
}

int ccdc_plan_tune_decode(ccdc_plan_t *p, int threads, int chunks) {
    if (!p) return CCDC_EINVAL;
    if (p->compression_mode || p->device != -1) return CCDC_ESTATE;
    if (chunks < 1 || chunks > p->nterm) return CCDC_EINVAL;
    const bool files = p->decode_files > 1;
    if (files ? threads != CCDC_DECODE_THREADS_FILES
              : (threads != CCDC_DECODE_THREADS && threads != CCDC_DECODE_THREADS_SHORT)) return CCDC_EINVAL;
    p->decode_threads = threads;
    set_split(*p, chunks);
    p->tuned = true;
    return CCDC_OK;
}

int ccdc_plan_kernel_family(const ccdc_plan_t *p) { return p ? p->family : 0; }

int ccdc_plan_tune_family(ccdc_plan_t *p, int family) {
    if (!p || (family != 0 && family != 1)) return CCDC_EINVAL;
    if (p->compression_mode || p->device != -1) return CCDC_ESTATE;
    const int before = p->family;
    p->family = family;
    ccdc_internal_choose_split(p);                  // the split follows the family's tile
    if (family == 1 && !ccdc_stream_supported(*p)) {
        p->family = before;
        ccdc_internal_choose_split(p);
        return CCDC_ESIZE;
    }
    p->family_tuned = true;
    return CCDC_OK;
}

int ccdc_plan_decode_threads(const ccdc_plan_t *p) { return p && !p->compression_mode ? p->decode_threads : 0; }
int ccdc_plan_decode_chunks(const ccdc_plan_t *p) { return p && !p->compression_mode ? p->nchunk : 0; }

long long ccdc_plan_num_jobs(const ccdc_plan_t *p) { return p ? p->J : 0; }
long long ccdc_plan_num_batches(const ccdc_plan_t *p) { return p ? p->nbatch : 0; }
long long ccdc_plan_num_groups(const ccdc_plan_t *p) { return p ? p->nround : 0; }
long long ccdc_plan_files_per_batch(const ccdc_plan_t *p) { return p ? p->b : 0; }
long long ccdc_plan_packet_elems(const ccdc_plan_t *p) { return p ? p->len : 0; }
long long ccdc_plan_segment_elems(const ccdc_plan_t *p) { return p ? p->s : 0; }
long long ccdc_plan_coded_row_elems(const ccdc_plan_t *p) { return p ? p->s_pad : 0; }
long long ccdc_plan_coded_bits(const ccdc_plan_t *p) {
    if (!p) return 0;
    if (p->compression_mode) return (long long)p->K * (p->nbatch - 1) * 32 * p->len;   // unicast packets
    return p->nround * (p->r + 1) * 32 * p->s;
}

int ccdc_plan_batch_of_file(const ccdc_plan_t *p, long long n, int *nodes_out) {
    if (!p || !nodes_out || n < 0 || n >= p->J * p->N) return CCDC_EINVAL;
    if (p->compression_mode) {      // holders of batch t: the nodes k with k mod m = t; padded with -1
        const long long t = std::min<long long>(n / p->b, p->nbatch - 1);
        int c = 0;
        for (int k = 0; k < p->K && c < p->r; ++k) if (k % p->nbatch == t) nodes_out[c++] = k;
        while (c < p->r) nodes_out[c++] = -1;
        return CCDC_OK;
    }
    const long long j = n / p->N, a = (n % p->N) / p->b;
    const long long b = p->job_batch0[j] + a;
    std::memcpy(nodes_out, &p->batch_nodes[(size_t)b * p->r], sizeof(int) * p->r);
    return CCDC_OK;
}

int ccdc_plan_batch(const ccdc_plan_t *p, long long b, int *nodes_out, long long *first_file, long long *job) {
    if (!p || b < 0 || b >= p->nbatch) return CCDC_EINVAL;
    if (p->compression_mode) {
        if (nodes_out) {
            int c = 0;
            for (int k = 0; k < p->K && c < p->r; ++k) if (k % p->nbatch == b) nodes_out[c++] = k;
            while (c < p->r) nodes_out[c++] = -1;
        }
        if (first_file) *first_file = p->batch_file0[b];
        if (job) *job = 0;
        return CCDC_OK;
    }
    if (nodes_out) std::memcpy(nodes_out, &p->batch_nodes[(size_t)b * p->r], sizeof(int) * p->r);
    if (first_file) *first_file = p->batch_file0[b];
    if (job) *job = p->batch_job[b];
    return CCDC_OK;
}

int ccdc_plan_group(const ccdc_plan_t *p, long long g, int *members_out) {
    if (!p || !members_out || g < 0 || g >= p->nround) return CCDC_EINVAL;
    std::memcpy(members_out, &p->round_group[(size_t)g * (p->r + 1)], sizeof(int) * (p->r + 1));
    return CCDC_OK;
}

int ccdc_plan_group_batches(const ccdc_plan_t *p, long long g, long long *batches_out) {
    if (!p || !batches_out || g < 0 || g >= p->nround) return CCDC_EINVAL;
    std::memcpy(batches_out, &p->round_batch[(size_t)g * (p->r + 1)], sizeof(long long) * (p->r + 1));
    return CCDC_OK;
}

long long ccdc_plan_node_batches(const ccdc_plan_t *p, int k, long long *ids_out) {
    if (!p || k < 0 || k >= p->K) return 0;
    if (ids_out) {
        long long n = 0;
        for (long long b = 0; b < p->nbatch; ++b)
            if (p->slot[(size_t)k * p->nbatch + b] >= 0) ids_out[n++] = b;
    }
    return p->nlocal[k];
}

size_t ccdc_partition_bytes(const ccdc_plan_t *p, int k) {
    if (!p || k < 0 || k >= p->K) return 0;
    return (size_t)(p->node_nfiles[k] * p->row_elems) * 4;
}

size_t ccdc_packets_bytes(const ccdc_plan_t *p, int k) {
    if (!p || k < 0 || k >= p->K) return 0;
    if (p->compression_mode) return 0;
    return (size_t)(p->nlocal[k] * (p->K - p->r) * p->len) * 4;
}

size_t ccdc_decoded_bytes(const ccdc_plan_t *p, int k) {
    if (!p || k < 0 || k >= p->K) return 0;
    return (size_t)(p->node_nrounds[k] * p->len) * 4;
}

size_t ccdc_coded_bytes(const ccdc_plan_t *p) {
    return p ? (size_t)(p->nround * (p->r + 1) * p->s_pad) * 4 : 0;
}

size_t ccdc_out_bytes(const ccdc_plan_t *p) { return p ? (size_t)(p->J * p->row_elems) * 4 : 0; }

int ccdc_plan_decode_cluster(const ccdc_plan_t *p) { return p && p->decode_cluster ? 1 : 0; }

size_t ccdc_workspace_bytes(const ccdc_plan_t *p) {
    if (!p || p->nchunk <= 1 || p->decode_cluster) return 0;
    return (size_t)p->nchunk * (size_t)(p->J * p->row_elems) * 4;
}

const char *ccdc_strerror(int status) {
    switch (status) {
    case CCDC_OK: return "ok";
    case CCDC_EINVAL: return "invalid argument (parameters outside the scheme's setting, NULL or misaligned pointer)";
    case CCDC_ENOMEM: return "out of memory";
    case CCDC_ECUDA: return "CUDA error (see ccdc_last_cuda_error)";
    case CCDC_ESIZE: return "size not supported by this entry point";
    case CCDC_ESTATE: return "call not valid for this plan";
    default: return "unknown status";
    }
}

}  // extern "C"
