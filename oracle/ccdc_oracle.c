/*
 * ccdc_oracle.c -- plain single-threaded CPU oracle for the compressed coded
 * distributed computing (compressed CDC) shuffle of Li, Maddah-Ali and
 * Avestimehr, "Compressed Coded Distributed Computing" (Section IV).
 *
 * THIS IS TEST INFRASTRUCTURE.  It exists so that the CUDA library can be
 * checked against something written directly from the paper.  It shares no
 * code with the library, is never called by the product path, and is slow on
 * purpose: every step is the paper's definition written out, node by node,
 * with one private memory per node and an explicit broadcast log.
 *
 * What each routine follows:
 *   placement          Section IV-A (batches labelled by size-muK subsets)
 *   function assignment Section III, "Shuffle phase" (the sets S_k)
 *   batch_sum/combine  Section IV-B, pre-combined value  vbar_{q,P}  and the
 *                      packet V_P obtained by concatenating Q/K of them
 *   segment            Section IV-B, V_P = (V_{P,i1}, ..., V_{P,i_muK})
 *   encode             Section IV-B, X_k = XOR over P containing k of V_{P,k}
 *                      (stage 1) and the same formula over batches of
 *                      different jobs (stage 2)
 *   decode             Section IV-B, cancellation of the segments V_{P,k'}
 *                      with k in P
 *   reduce             Eq. (1) and the final reduction paragraph of Section IV
 *   bit counter        Definition 1 (communication load)
 *
 * Two plans are offered.  "single": one job whose N files are spread over
 * all C(K,r) size-r subsets of the K nodes and one multicast round per
 * size-(r+1) subset.  "paper": the scheme exactly as Section IV states it,
 * J = C(K,r+1) jobs, job j living on its own (r+1)-subset, K-r rounds per
 * subset (stage 1 plus one stage-2 round per outside node).  Inside a round
 * both run the same routines below.
 *
 * Parity status: every routine here is pinned by tests/test_oracle_pins.py
 * (brute force of Eq. (1), the decode invariant, the paper's printed loads
 * for its two worked examples, Theorem 1, closed forms).  The one reading
 * that the paper cannot pin is the treatment of a packet whose length is not
 * a multiple of r (equal segments of ceil(len/r) words, zero extended):
 * "parity unpinned" for that reading only.
 *
 * Arithmetic: 32-bit words.  dtype 0 = int32 with wrapping addition,
 * dtype 1 = IEEE binary32 addition (compile with -ffp-contract=off and
 * without -ffast-math).  XOR always acts on the raw 32-bit patterns.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

#define ORACLE_MAX_K 64

enum { ORACLE_I32 = 0, ORACLE_F32 = 1 };

typedef struct ccdc_oracle {
    int K, r, Q, dtype, paper_mode;
    int64_t N;          /* files per job */
    int64_t B;          /* 32-bit elements per intermediate value (T = 32 B bits) */
    int64_t J;          /* jobs */
    int64_t b;          /* files per batch */
    int64_t len;        /* words per packet V_P: (Q/K) * B */
    int64_t s;          /* words per segment: ceil(len / r) */
    int64_t nbatch;     /* batches over all jobs */
    int64_t nround;     /* multicast rounds */
    int *batch_nodes;       /* [nbatch][r], ascending: the label P of the batch */
    int64_t *batch_file0;   /* [nbatch] first global file id (job*N + n) */
    int64_t *batch_job;     /* [nbatch] */
    int *round_group;       /* [nround][r+1], ascending: the subset of nodes */
    int64_t *round_batch;   /* [nround][r+1]: batch whose packet member a must receive */
    int64_t *recv_round;    /* [nbatch][K]: round in which node k receives batch p, or -1 */
    /* one private memory per node: [local batch][file in batch][q][B] */
    uint32_t *mem[ORACLE_MAX_K];
    int64_t *slot[ORACLE_MAX_K];    /* [nbatch] local index of batch p at node k, or -1 */
    int64_t nlocal[ORACLE_MAX_K];
    /* broadcast medium: every coded packet, in the order it was sent */
    uint32_t *log;          /* [nround][r+1][s] */
    int64_t log_bits;
    uint32_t *decoded;      /* [nround][r+1][len]: what member a recovered */
    int loaded, shuffled;
} ccdc_oracle;

/* ------------------------------------------------------------------ */
/* small combinatorics                                                 */

static int64_t binom(int n, int k)
{
    if (k < 0 || k > n) return 0;
    if (k > n - k) k = n - k;
    int64_t c = 1;
    for (int i = 1; i <= k; ++i) {
        /* c * (n-k+i) / i is exact at every step */
        if (c > INT64_MAX / (n - k + i)) return -1;
        c = c * (n - k + i) / i;
    }
    return c;
}

static void first_subset(int *c, int m)
{
    for (int i = 0; i < m; ++i) c[i] = i;
}

/* next m-subset of {0..n-1} in lexicographic order; 0 when exhausted */
static int next_subset(int *c, int m, int n)
{
    int i = m - 1;
    while (i >= 0 && c[i] == n - m + i) --i;
    if (i < 0) return 0;
    ++c[i];
    for (int j = i + 1; j < m; ++j) c[j] = c[j - 1] + 1;
    return 1;
}

static int contains(const int *set, int m, int x)
{
    for (int i = 0; i < m; ++i) if (set[i] == x) return 1;
    return 0;
}

/* position of x inside the ascending set (its segment label index), or -1 */
static int label_index(const int *set, int m, int x)
{
    for (int i = 0; i < m; ++i) if (set[i] == x) return i;
    return -1;
}

/* batch of job `job` whose label is exactly `nodes` (r ascending ids), or -1 */
static int64_t find_batch(const ccdc_oracle *o, int64_t job, const int *nodes)
{
    for (int64_t p = 0; p < o->nbatch; ++p) {
        if (o->batch_job[p] != job) continue;
        if (memcmp(o->batch_nodes + p * o->r, nodes, sizeof(int) * (size_t)o->r) == 0) return p;
    }
    return -1;
}

/* S without its a-th member */
static void drop_member(const int *S, int m, int a, int *out)
{
    int n = 0;
    for (int i = 0; i < m; ++i) if (i != a) out[n++] = S[i];
}

/* ------------------------------------------------------------------ */
/* construction                                                        */

void oracle_free(ccdc_oracle *o)
{
    if (!o) return;
    free(o->batch_nodes); free(o->batch_file0); free(o->batch_job);
    free(o->round_group); free(o->round_batch); free(o->recv_round);
    for (int k = 0; k < ORACLE_MAX_K; ++k) { free(o->mem[k]); free(o->slot[k]); }
    free(o->log); free(o->decoded);
    free(o);
}

static ccdc_oracle *alloc_common(int K, int r, int64_t N, int Q, int64_t B, int dtype)
{
    if (K < 2 || K > ORACLE_MAX_K) return NULL;
    if (r < 1 || r > K - 1) return NULL;           /* mu K in {1..K-1} (Theorem 1) */
    if (N < K) return NULL;                        /* K <= N (network model) */
    if (Q < K || Q % K != 0) return NULL;          /* K | Q (network model) */
    if (B < 1) return NULL;
    if (dtype != ORACLE_I32 && dtype != ORACLE_F32) return NULL;
    ccdc_oracle *o = (ccdc_oracle *)calloc(1, sizeof(*o));
    if (!o) return NULL;
    o->K = K; o->r = r; o->N = N; o->Q = Q; o->B = B; o->dtype = dtype;
    o->len = (int64_t)(Q / K) * B;
    o->s = (o->len + r - 1) / r;
    return o;
}

/* fill recv_round from the rounds and check that every batch reaches every
 * outside node exactly once and that each round has the structure Section IV
 * prescribes (the batch meant for member t is labelled by the group minus t) */
static int finish_plan(ccdc_oracle *o)
{
    const int r = o->r, K = o->K;
    o->recv_round = (int64_t *)malloc(sizeof(int64_t) * (size_t)(o->nbatch * K));
    if (!o->recv_round) return -1;
    for (int64_t i = 0; i < o->nbatch * K; ++i) o->recv_round[i] = -1;
    int rest[ORACLE_MAX_K];
    for (int64_t ro = 0; ro < o->nround; ++ro) {
        const int *S = o->round_group + ro * (r + 1);
        for (int a = 0; a <= r; ++a) {
            int64_t p = o->round_batch[ro * (r + 1) + a];
            if (p < 0 || p >= o->nbatch) return -2;
            drop_member(S, r + 1, a, rest);
            if (memcmp(rest, o->batch_nodes + p * r, sizeof(int) * (size_t)r) != 0) return -3;
            if (o->recv_round[p * K + S[a]] != -1) return -4;     /* delivered twice */
            o->recv_round[p * K + S[a]] = ro;
        }
    }
    for (int64_t p = 0; p < o->nbatch; ++p)
        for (int k = 0; k < K; ++k) {
            int inside = contains(o->batch_nodes + p * r, r, k);
            if (inside && o->recv_round[p * K + k] != -1) return -5;
            if (!inside && o->recv_round[p * K + k] == -1) return -6;  /* never delivered */
        }
    /* node storage */
    for (int k = 0; k < K; ++k) {
        o->slot[k] = (int64_t *)malloc(sizeof(int64_t) * (size_t)o->nbatch);
        if (!o->slot[k]) return -1;
        int64_t n = 0;
        for (int64_t p = 0; p < o->nbatch; ++p)
            o->slot[k][p] = contains(o->batch_nodes + p * r, r, k) ? n++ : -1;
        o->nlocal[k] = n;
    }
    return 0;
}

/* One job over all K nodes: batch p is labelled by the p-th size-r subset of
 * {0..K-1} (lexicographic) and holds files p*b .. p*b+b-1; one round per
 * size-(r+1) subset S, in which member t receives the batch labelled S\{t}. */
ccdc_oracle *oracle_new_single(int K, int r, int64_t N, int Q, int64_t B, int dtype)
{
    ccdc_oracle *o = alloc_common(K, r, N, Q, B, dtype);
    if (!o) return NULL;
    int64_t nb = binom(K, r), ng = binom(K, r + 1);
    if (nb <= 0 || ng <= 0 || N % nb != 0) { oracle_free(o); return NULL; }
    o->paper_mode = 0; o->J = 1; o->b = N / nb; o->nbatch = nb; o->nround = ng;
    o->batch_nodes = (int *)malloc(sizeof(int) * (size_t)(nb * r));
    o->batch_file0 = (int64_t *)malloc(sizeof(int64_t) * (size_t)nb);
    o->batch_job = (int64_t *)calloc((size_t)nb, sizeof(int64_t));
    o->round_group = (int *)malloc(sizeof(int) * (size_t)(ng * (r + 1)));
    o->round_batch = (int64_t *)malloc(sizeof(int64_t) * (size_t)(ng * (r + 1)));
    if (!o->batch_nodes || !o->batch_file0 || !o->batch_job || !o->round_group || !o->round_batch) {
        oracle_free(o); return NULL;
    }
    int c[ORACLE_MAX_K], rest[ORACLE_MAX_K];
    int64_t p = 0;
    first_subset(c, r);
    do {
        memcpy(o->batch_nodes + p * r, c, sizeof(int) * (size_t)r);
        o->batch_file0[p] = p * o->b;
        ++p;
    } while (next_subset(c, r, K));
    int64_t g = 0;
    first_subset(c, r + 1);
    do {
        memcpy(o->round_group + g * (r + 1), c, sizeof(int) * (size_t)(r + 1));
        for (int a = 0; a <= r; ++a) {
            drop_member(c, r + 1, a, rest);
            o->round_batch[g * (r + 1) + a] = find_batch(o, 0, rest);
        }
        ++g;
    } while (next_subset(c, r + 1, K));
    if (finish_plan(o) != 0) { oracle_free(o); return NULL; }
    return o;
}

/* The scheme as Section IV states it, gamma = 1: job j lives on the j-th
 * size-(r+1) subset K_j; its N files are cut into r+1 equal batches labelled
 * by the size-r subsets of K_j.  Rounds, per subset S = K_j: stage 1 (all
 * batches of job j), then for each outside node i one stage-2 round in which
 * member t receives the batch labelled S\{t} of the job living on
 * {i} U S\{t}. */
ccdc_oracle *oracle_new_paper(int K, int r, int64_t N, int Q, int64_t B, int dtype)
{
    ccdc_oracle *o = alloc_common(K, r, N, Q, B, dtype);
    if (!o) return NULL;
    int64_t J = binom(K, r + 1);
    if (J <= 0 || N % (r + 1) != 0) { oracle_free(o); return NULL; }
    o->paper_mode = 1; o->J = J; o->b = N / (r + 1);
    o->nbatch = J * (r + 1);
    o->nround = J * (K - r);
    int64_t nb = o->nbatch, nr = o->nround;
    o->batch_nodes = (int *)malloc(sizeof(int) * (size_t)(nb * r));
    o->batch_file0 = (int64_t *)malloc(sizeof(int64_t) * (size_t)nb);
    o->batch_job = (int64_t *)malloc(sizeof(int64_t) * (size_t)nb);
    o->round_group = (int *)malloc(sizeof(int) * (size_t)(nr * (r + 1)));
    o->round_batch = (int64_t *)malloc(sizeof(int64_t) * (size_t)(nr * (r + 1)));
    int *job_nodes = (int *)malloc(sizeof(int) * (size_t)(J * (r + 1)));
    if (!o->batch_nodes || !o->batch_file0 || !o->batch_job || !o->round_group ||
        !o->round_batch || !job_nodes) { free(job_nodes); oracle_free(o); return NULL; }
    int c[ORACLE_MAX_K], d[ORACLE_MAX_K], rest[ORACLE_MAX_K], home[ORACLE_MAX_K];
    int64_t j = 0, p = 0;
    first_subset(c, r + 1);
    do {
        memcpy(job_nodes + j * (r + 1), c, sizeof(int) * (size_t)(r + 1));
        /* the r+1 size-r subsets of K_j in lexicographic order */
        int64_t a = 0;
        first_subset(d, r);
        do {
            for (int i = 0; i < r; ++i) o->batch_nodes[p * r + i] = c[d[i]];
            o->batch_job[p] = j;
            o->batch_file0[p] = j * N + a * o->b;
            ++p; ++a;
        } while (next_subset(d, r, r + 1));
        ++j;
    } while (next_subset(c, r + 1, K));
    int64_t ro = 0;
    for (j = 0; j < J; ++j) {
        const int *S = job_nodes + j * (r + 1);
        /* stage 1 */
        memcpy(o->round_group + ro * (r + 1), S, sizeof(int) * (size_t)(r + 1));
        for (int a = 0; a <= r; ++a) {
            drop_member(S, r + 1, a, rest);
            o->round_batch[ro * (r + 1) + a] = find_batch(o, j, rest);
        }
        ++ro;
        /* stage 2, one round per outside node i */
        for (int i = 0; i < K; ++i) {
            if (contains(S, r + 1, i)) continue;
            memcpy(o->round_group + ro * (r + 1), S, sizeof(int) * (size_t)(r + 1));
            for (int a = 0; a <= r; ++a) {
                drop_member(S, r + 1, a, rest);
                /* home = {i} U S\{t}, ascending */
                int n = 0, placed = 0;
                for (int x = 0; x < r; ++x) {
                    if (!placed && i < rest[x]) { home[n++] = i; placed = 1; }
                    home[n++] = rest[x];
                }
                if (!placed) home[n++] = i;
                int64_t jt = -1;
                for (int64_t jj = 0; jj < J; ++jj)
                    if (memcmp(job_nodes + jj * (r + 1), home, sizeof(int) * (size_t)(r + 1)) == 0) jt = jj;
                o->round_batch[ro * (r + 1) + a] = (jt < 0) ? -1 : find_batch(o, jt, rest);
            }
            ++ro;
        }
    }
    free(job_nodes);
    if (ro != nr || finish_plan(o) != 0) { oracle_free(o); return NULL; }
    return o;
}

/* ------------------------------------------------------------------ */
/* queries                                                             */

int64_t oracle_num_jobs(const ccdc_oracle *o) { return o->J; }
int64_t oracle_num_batches(const ccdc_oracle *o) { return o->nbatch; }
int64_t oracle_num_rounds(const ccdc_oracle *o) { return o->nround; }
int64_t oracle_files_per_batch(const ccdc_oracle *o) { return o->b; }
int64_t oracle_packet_elems(const ccdc_oracle *o) { return o->len; }
int64_t oracle_segment_elems(const ccdc_oracle *o) { return o->s; }
int64_t oracle_node_num_batches(const ccdc_oracle *o, int k) { return o->nlocal[k]; }
int64_t oracle_batch_job(const ccdc_oracle *o, int64_t p) { return o->batch_job[p]; }
int64_t oracle_batch_first_file(const ccdc_oracle *o, int64_t p) { return o->batch_file0[p]; }
int64_t oracle_recv_round(const ccdc_oracle *o, int64_t p, int k) { return o->recv_round[p * o->K + k]; }

void oracle_batch_nodes(const ccdc_oracle *o, int64_t p, int *out)
{
    memcpy(out, o->batch_nodes + p * o->r, sizeof(int) * (size_t)o->r);
}

void oracle_round_group(const ccdc_oracle *o, int64_t ro, int *out)
{
    memcpy(out, o->round_group + ro * (o->r + 1), sizeof(int) * (size_t)(o->r + 1));
}

void oracle_round_batches(const ccdc_oracle *o, int64_t ro, int64_t *out)
{
    memcpy(out, o->round_batch + ro * (o->r + 1), sizeof(int64_t) * (size_t)(o->r + 1));
}

/* ------------------------------------------------------------------ */
/* Map output placement: node k receives a private copy of v_{q,n} for
 * every file n it stores and every q (Section III, Map phase).
 * v is [J*N files][Q][B] words.                                        */

int oracle_load_values(ccdc_oracle *o, const uint32_t *v)
{
    const int64_t row = (int64_t)o->Q * o->B;
    for (int k = 0; k < o->K; ++k) {
        free(o->mem[k]);
        size_t words = (size_t)(o->nlocal[k] * o->b * row);
        o->mem[k] = (uint32_t *)malloc(sizeof(uint32_t) * (words ? words : 1));
        if (!o->mem[k]) return -1;
        for (int64_t p = 0; p < o->nbatch; ++p) {
            int64_t sl = o->slot[k][p];
            if (sl < 0) continue;
            for (int64_t f = 0; f < o->b; ++f)
                memcpy(o->mem[k] + (sl * o->b + f) * row,
                       v + (o->batch_file0[p] + f) * row, sizeof(uint32_t) * (size_t)row);
        }
    }
    o->loaded = 1; o->shuffled = 0;
    return 0;
}

/* ------------------------------------------------------------------ */
/* arithmetic                                                          */

static uint32_t add_words(int dtype, uint32_t a, uint32_t b)
{
    if (dtype == ORACLE_I32) return a + b;              /* wraps mod 2^32 */
    float x, y, z;
    memcpy(&x, &a, 4); memcpy(&y, &b, 4);
    z = x + y;                                          /* binary32, round to nearest even */
    uint32_t w; memcpy(&w, &z, 4);
    return w;
}

/* vbar_{q,P}[e] at node k: the files of the batch in ascending order, left to
 * right, starting from the first file's value (so a one-file batch passes
 * its bits through unchanged). */
static uint32_t batch_sum(const ccdc_oracle *o, int k, int64_t p, int q, int64_t e)
{
    const int64_t sl = o->slot[k][p];            /* caller guarantees sl >= 0 */
    const uint32_t *base = o->mem[k] + (sl * o->b) * (int64_t)o->Q * o->B;
    uint32_t acc = base[(int64_t)q * o->B + e];
    for (int64_t f = 1; f < o->b; ++f)
        acc = add_words(o->dtype, acc, base[(f * o->Q + q) * o->B + e]);
    return acc;
}

/* packet V_P meant for node t, built at node k (k in P): the Q/K pre-combined
 * values of t's functions, ascending q, concatenated */
static void combine(const ccdc_oracle *o, int k, int64_t p, int t, uint32_t *out)
{
    const int per = o->Q / o->K;
    for (int c = 0; c < per; ++c)
        for (int64_t e = 0; e < o->B; ++e)
            out[(int64_t)c * o->B + e] = batch_sum(o, k, p, t * per + c, e);
}

/* i-th of the r equal segments of a packet, zero extended to s words */
static void segment(const ccdc_oracle *o, const uint32_t *packet, int i, uint32_t *out)
{
    for (int64_t j = 0; j < o->s; ++j) {
        int64_t idx = (int64_t)i * o->s + j;
        out[j] = idx < o->len ? packet[idx] : 0u;
    }
}

/* ------------------------------------------------------------------ */
/* shuffle: every round's encode, broadcast, decode                    */

/* encode of one round at every member k' = S[as]: the XOR of the segments
 * labelled k' of the r packets k' has built; appended to the broadcast log */
static void encode_round(ccdc_oracle *o, int64_t ro, uint32_t *pkt, uint32_t *seg)
{
    const int r = o->r;
    const int64_t s = o->s;
    const int *S = o->round_group + ro * (r + 1);
    const int64_t *bat = o->round_batch + ro * (r + 1);
    for (int as = 0; as <= r; ++as) {
        const int ks = S[as];
        uint32_t *x = o->log + (ro * (r + 1) + as) * s;
        memset(x, 0, sizeof(uint32_t) * (size_t)s);
        for (int a = 0; a <= r; ++a) {
            if (a == as) continue;
            combine(o, ks, bat[a], S[a], pkt);
            segment(o, pkt, label_index(o->batch_nodes + bat[a] * r, r, ks), seg);
            for (int64_t j = 0; j < s; ++j) x[j] ^= seg[j];
        }
        o->log_bits += 32 * s;      /* one broadcast, counted once */
    }
}

/* decode of one round at every member k = S[ak], from the log and k's own
 * memory only; returns 0, -10 or -11 (see oracle_shuffle) */
static int decode_round(ccdc_oracle *o, int64_t ro, uint32_t *pkt, uint32_t *seg, uint32_t *y)
{
    const int r = o->r;
    const int64_t s = o->s, len = o->len;
    const int *S = o->round_group + ro * (r + 1);
    const int64_t *bat = o->round_batch + ro * (r + 1);
    int rc = 0;
    for (int ak = 0; ak <= r; ++ak) {
        const int k = S[ak];
        uint32_t *rec = o->decoded + (ro * (r + 1) + ak) * len;
        for (int as = 0; as <= r; ++as) {
            if (as == ak) continue;
            const int ks = S[as];
            memcpy(y, o->log + (ro * (r + 1) + as) * s, sizeof(uint32_t) * (size_t)s);
            for (int a = 0; a <= r; ++a) {
                if (a == ak || a == as) continue;
                combine(o, k, bat[a], S[a], pkt);
                segment(o, pkt, label_index(o->batch_nodes + bat[a] * r, r, ks), seg);
                for (int64_t j = 0; j < s; ++j) y[j] ^= seg[j];
            }
            const int i0 = label_index(o->batch_nodes + bat[ak] * r, r, ks);
            for (int64_t j = 0; j < s; ++j) {
                int64_t idx = (int64_t)i0 * s + j;
                if (idx < len) rec[idx] = y[j];
                else if (y[j] != 0u) rc = -11;
            }
        }
        /* test-only check with the senders' copies: what k recovered is the
         * packet every node of the batch built */
        for (int i = 0; i < r; ++i) {
            combine(o, o->batch_nodes[bat[ak] * r + i], bat[ak], k, pkt);
            if (memcmp(pkt, rec, sizeof(uint32_t) * (size_t)len) != 0) rc = -10;
        }
    }
    return rc;
}

/* The Shuffle phase, round by round: encode, broadcast, decode.
 * returns 0, or a negative code: -1 memory, -2 not loaded,
 * -10 a receiver failed to recover its packet bit for bit,
 * -11 a decoded zero extension was not zero.
 * With decode_only != 0 the log is kept as it is and only the decodes run
 * (used by tests that damage a broadcast packet). */
static int shuffle_impl(ccdc_oracle *o, int decode_only)
{
    if (!o->loaded) return -2;
    if (decode_only && !o->log) return -2;
    const int r = o->r;
    const int64_t s = o->s, len = o->len;
    if (!decode_only) {
        free(o->log); free(o->decoded);
        o->log = (uint32_t *)calloc((size_t)(o->nround * (r + 1) * s) + 1, sizeof(uint32_t));
        o->decoded = (uint32_t *)calloc((size_t)(o->nround * (r + 1) * len) + 1, sizeof(uint32_t));
        o->log_bits = 0;
    }
    uint32_t *pkt = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)len);
    uint32_t *seg = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)s);
    uint32_t *y = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)s);
    int rc = 0;
    if (!o->log || !o->decoded || !pkt || !seg || !y) { rc = -1; goto done; }
    for (int64_t ro = 0; ro < o->nround; ++ro) {
        if (!decode_only) encode_round(o, ro, pkt, seg);
        int e = decode_round(o, ro, pkt, seg, y);
        if (e != 0) rc = e;
    }
    o->shuffled = (rc == 0);
done:
    free(pkt); free(seg); free(y);
    return rc;
}

int oracle_shuffle(ccdc_oracle *o) { return shuffle_impl(o, 0); }
int oracle_redecode(ccdc_oracle *o) { return shuffle_impl(o, 1); }

/* fault planting for the tests: flip bits of one word of node k's private
 * memory, or of one word of the broadcast log */
void oracle_poke_node(ccdc_oracle *o, int k, int64_t word, uint32_t mask) { o->mem[k][word] ^= mask; }
void oracle_poke_log(ccdc_oracle *o, int64_t word, uint32_t mask) { o->log[word] ^= mask; }

int64_t oracle_coded_bits(const ccdc_oracle *o) { return o->log_bits; }

/* copy of the broadcast log, [round][sender rank in the group][s] */
void oracle_copy_coded(const ccdc_oracle *o, uint32_t *out)
{
    memcpy(out, o->log, sizeof(uint32_t) * (size_t)(o->nround * (o->r + 1) * o->s));
}

/* packets node k builds, [local batch][outside node t ascending][len] */
void oracle_copy_packets(const ccdc_oracle *o, int k, uint32_t *out)
{
    int64_t n = 0;
    for (int64_t p = 0; p < o->nbatch; ++p) {
        if (o->slot[k][p] < 0) continue;
        for (int t = 0; t < o->K; ++t) {
            if (contains(o->batch_nodes + p * o->r, o->r, t)) continue;
            combine(o, k, p, t, out + n * o->len);
            ++n;
        }
    }
}

/* packets node k recovered, in round order, [round containing k][len] */
void oracle_copy_decoded(const ccdc_oracle *o, int k, uint32_t *out)
{
    int64_t n = 0;
    for (int64_t ro = 0; ro < o->nround; ++ro) {
        int a = label_index(o->round_group + ro * (o->r + 1), o->r + 1, k);
        if (a < 0) continue;
        memcpy(out + n * o->len, o->decoded + (ro * (o->r + 1) + a) * o->len,
               sizeof(uint32_t) * (size_t)o->len);
        ++n;
    }
}

/* ------------------------------------------------------------------ */
/* Reduce (Eq. (1)): node k, function q of job j.  Batches of the job in
 * ascending order; a batch k stores contributes its local pre-combined
 * value, any other batch the value k decoded.  out is [J*Q][B] words.   */

int oracle_reduce(const ccdc_oracle *o, uint32_t *out)
{
    if (!o->shuffled) return -2;
    const int per = o->Q / o->K;
    for (int64_t j = 0; j < o->J; ++j)
        for (int k = 0; k < o->K; ++k)
            for (int c = 0; c < per; ++c) {
                const int q = k * per + c;
                uint32_t *dst = out + (j * o->Q + q) * o->B;
                for (int64_t e = 0; e < o->B; ++e) {
                    uint32_t acc = 0u;
                    for (int64_t p = 0; p < o->nbatch; ++p) {
                        if (o->batch_job[p] != j) continue;
                        uint32_t term;
                        if (o->slot[k][p] >= 0) {
                            term = batch_sum(o, k, p, q, e);
                        } else {
                            int64_t ro = o->recv_round[p * o->K + k];
                            int a = label_index(o->round_group + ro * (o->r + 1), o->r + 1, k);
                            term = o->decoded[(ro * (o->r + 1) + a) * o->len + (int64_t)c * o->B + e];
                        }
                        acc = add_words(o->dtype, acc, term);
                    }
                    dst[e] = acc;
                }
            }
    return 0;
}

/* ------------------------------------------------------------------ */
/* Direct evaluation of Eq. (1) from the values themselves (no scheme):
 * int32: wrapped sum.  fp32: sum and sum of magnitudes in binary64.    */

void oracle_direct_i32(const ccdc_oracle *o, const uint32_t *v, uint32_t *out)
{
    for (int64_t j = 0; j < o->J; ++j)
        for (int q = 0; q < o->Q; ++q)
            for (int64_t e = 0; e < o->B; ++e) {
                uint32_t acc = 0u;
                for (int64_t n = 0; n < o->N; ++n)
                    acc += v[((j * o->N + n) * o->Q + q) * o->B + e];
                out[(j * o->Q + q) * o->B + e] = acc;
            }
}

void oracle_direct_f64(const ccdc_oracle *o, const uint32_t *v, double *sum, double *abs_sum)
{
    for (int64_t j = 0; j < o->J; ++j)
        for (int q = 0; q < o->Q; ++q)
            for (int64_t e = 0; e < o->B; ++e) {
                double a = 0.0, m = 0.0;
                for (int64_t n = 0; n < o->N; ++n) {
                    float x;
                    memcpy(&x, &v[((j * o->N + n) * o->Q + q) * o->B + e], 4);
                    a += (double)x; m += fabs((double)x);
                }
                sum[(j * o->Q + q) * o->B + e] = a;
                abs_sum[(j * o->Q + q) * o->B + e] = m;
            }
}

/* ------------------------------------------------------------------ */
/* Bits other shuffles would broadcast on the SAME placement, counted by
 * enumeration (Definition 1 counts every broadcast once):
 *  uncoded    every node is sent, value by value, what it does not store
 *  combining  every node is sent one pre-combined packet per batch it does
 *             not store (Section II, compression scheme)
 *  plain CDC  the same rounds, but coded file by file without pre-combining
 *             (Section II, CDC scheme)                                  */

int64_t oracle_bits_uncoded(const ccdc_oracle *o)
{
    int64_t bits = 0;
    for (int k = 0; k < o->K; ++k)
        for (int64_t p = 0; p < o->nbatch; ++p)
            if (o->slot[k][p] < 0) bits += o->b * 32 * o->len;
    return bits;
}

int64_t oracle_bits_combining(const ccdc_oracle *o)
{
    int64_t bits = 0;
    for (int k = 0; k < o->K; ++k)
        for (int64_t p = 0; p < o->nbatch; ++p)
            if (o->slot[k][p] < 0) bits += 32 * o->len;
    return bits;
}

int64_t oracle_bits_plain_cdc(const ccdc_oracle *o)
{
    int64_t bits = 0;
    for (int64_t ro = 0; ro < o->nround; ++ro)
        for (int as = 0; as <= o->r; ++as)
            for (int64_t f = 0; f < o->b; ++f) bits += 32 * o->s;
    return bits;
}

/* files stored at node k (storage constraint of Section III) */
int64_t oracle_node_num_files(const ccdc_oracle *o, int k) { return o->nlocal[k] * o->b; }

/* ------------------------------------------------------------------ */
/* Compression-only scheme (Appendix, "Communication Load of the compression
 * scheme"), one job.  The files are cut into m = ceil(1/mu) batches: the first
 * m-1 hold mu*N files each, the last one the rest; node k stores batch k mod m
 * (0-based).  For every function of node k and every batch t it does not store,
 * one node that stores batch t pre-combines the batch for that function and
 * unicasts the packet to k; k adds the m-1 packets to its own batch sum.
 * The paper leaves the choice of the sender open; here it is the first node
 * after k, cyclically, that stores batch t.
 *
 * v     [N][Q][B] words, mu = r/K (K | r*N required)
 * out   [Q][B]
 * recv  [K][m-1][len]: packets node k received, batches ascending
 * returns the number of bits sent (every unicast counted once, Definition 1),
 * or -1 on invalid parameters / memory.                                   */
int64_t oracle_compression_run(int K, int r, int64_t N, int Q, int64_t B, int dtype,
                               const uint32_t *v, uint32_t *out, uint32_t *recv,
                               int64_t *files_at_node /* [K] */)
{
    if (K < 2 || r < 1 || r > K - 1 || N < K || Q % K != 0 || B < 1) return -1;
    if ((r * N) % K != 0) return -1;
    const int m = (K + r - 1) / r;                   /* ceil(1/mu) */
    const int64_t full = r * N / K;                  /* mu*N files in the first m-1 batches */
    const int64_t last = N - (int64_t)(m - 1) * full;
    if (last < 1) return -1;
    const int per = Q / K;
    const int64_t len = (int64_t)per * B, row = (int64_t)Q * B;
    uint32_t **mem = (uint32_t **)calloc((size_t)K, sizeof(uint32_t *));
    if (!mem) return -1;
    int64_t bits = 0;
    /* placement: node k holds a private copy of batch k mod m */
    for (int k = 0; k < K; ++k) {
        const int t = k % m;
        const int64_t nf = t == m - 1 ? last : full;
        mem[k] = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)(nf * row));
        if (!mem[k]) { bits = -1; goto done; }
        memcpy(mem[k], v + (int64_t)t * full * row, sizeof(uint32_t) * (size_t)(nf * row));
        if (files_at_node) files_at_node[k] = nf;
    }
    /* shuffle: unicast of pre-combined packets */
    for (int k = 0; k < K; ++k) {
        int slot = 0;
        for (int t = 0; t < m; ++t) {
            if (t == k % m) continue;
            int ks = (k + 1) % K;
            while (ks % m != t) ks = (ks + 1) % K;   /* first node after k that stores batch t */
            const int64_t nf = t == m - 1 ? last : full;
            uint32_t *pkt = recv + ((int64_t)k * (m - 1) + slot) * len;
            for (int c = 0; c < per; ++c)
                for (int64_t e = 0; e < B; ++e) {
                    const int q = k * per + c;
                    uint32_t acc = mem[ks][(int64_t)q * B + e];
                    for (int64_t f = 1; f < nf; ++f)
                        acc = add_words(dtype, acc, mem[ks][(f * Q + q) * B + e]);
                    pkt[(int64_t)c * B + e] = acc;
                }
            bits += 32 * len;
            ++slot;
        }
    }
    /* reduce at node k: batches ascending, own batch from own memory */
    for (int k = 0; k < K; ++k)
        for (int c = 0; c < per; ++c)
            for (int64_t e = 0; e < B; ++e) {
                const int q = k * per + c;
                uint32_t acc = 0u;
                int slot = 0;
                for (int t = 0; t < m; ++t) {
                    uint32_t term;
                    if (t == k % m) {
                        const int64_t nf = t == m - 1 ? last : full;
                        term = mem[k][(int64_t)q * B + e];
                        for (int64_t f = 1; f < nf; ++f)
                            term = add_words(dtype, term, mem[k][(f * Q + q) * B + e]);
                    } else {
                        term = recv[((int64_t)k * (m - 1) + slot) * len + (int64_t)c * B + e];
                        ++slot;
                    }
                    acc = add_words(dtype, acc, term);
                }
                out[(int64_t)q * B + e] = acc;
            }
done:
    for (int k = 0; k < K; ++k) free(mem[k]);
    free(mem);
    return bits;
}
