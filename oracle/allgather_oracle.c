/*
 * CPU oracle for the allgather schedules of the Sparbit paper.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain statement of what the step executor must compute.  It is used by
 * the tests, by the smoke check and by the benchmark's CPU-baseline leg; the product (the CUDA
 * library) neither links nor calls it, and it shares no code, header or table with the product.
 *
 * What it does
 * ------------
 * P simulated MPI ranks each own one send block (m bytes) and one receive buffer of P slots
 * (Section II: after the call, slot j of every receive buffer holds the block sent by rank j).
 * For a chosen algorithm every rank, on its own, posts the sends and receives the algorithm
 * prescribes for every step (explicit lists, one entry per block, as Algorithm 1 issues one
 * MPI_Isend and one MPI_Irecv per block).  The lists of all ranks are then matched the way MPI
 * matches point-to-point traffic (the k-th send from a to b meets the k-th receive that b posted
 * for a), checked, and flattened into one message list ordered by phase.  Running the collective
 * is then one memcpy per message, a phase at a time.
 *
 * Phases: -1 is the local copy of the own send block into the receive buffer (Algorithm 1 sends
 * displacement `rank` at j = 0 as if it were already there; the MPI semantics of Section II need
 * the copy).  0..K-1 are the algorithm's communication steps.  Bruck has one more local phase, K,
 * the final rotation ("memory shifts", Section II-B).
 *
 * Algorithms
 * ----------
 *   SPARBIT  Algorithm 1 of the paper, statement by statement.
 *   RING     Section II-A: p-1 steps, r -> r+1, own block first, then forward what arrived last.
 *   RD       Section II-A recursive doubling: log2 p steps, partner r xor 2^s, send all held;
 *            defined for powers of two only (the paper states the restriction).
 *   NE       Section II-A neighbor exchange: p/2 steps, even p only; on step s an even rank r
 *            exchanges with r + (-1)^s and an odd rank with r - (-1)^s (wrap-around); one block
 *            (the own) on the first step, two blocks on every other step.  Which two the paper
 *            leaves open; the reading taken: on step 1 a rank sends the two blocks it holds,
 *            on every later step the two blocks it received on the previous step (the ring's
 *            rule, applied pairwise).  A rank receives what its partner sends.
 *   BRUCK    Section II-A: floor(log2 p) steps sending everything held to r - 2^s, receiving
 *            from r + 2^s, one more step with the first p - 2^floor(log2 p) blocks when p is
 *            not a power of two, then the rotation.  Local order: slot i of the working buffer
 *            of rank r holds the block of rank (r + i) mod p.
 *
 * Checks made while the plan is built (any failure makes plan creation fail with a message):
 *   - posted send and receive lists of every ordered pair have equal length per step;
 *   - a message reads only a location that was valid when the phase began, and writes only a
 *     location that is neither valid nor already written in this phase (so the read set and the
 *     write set of a phase are disjoint and in-place execution equals snapshot execution);
 *   - for SPARBIT, RING and RD the sender's and the receiver's displacement agree;
 *   - the identity of the block carried into receive slot b is b, every receive slot is written
 *     exactly once, and every rank receives exactly P-1 blocks from other ranks.
 *
 * Parity status: pinned (see the CPU tests: plain definition of the result for all five
 * algorithms, the paper's P = 5 walk-through, the P = 21 decomposition, an independent
 * binomial-tree construction, closed forms, the partner rule and block counts of the neighbor
 * exchange, brute force over P = 1..64; for the variable-size runs the plain definition with
 * byte-granular sizes including empty blocks, and equality with the fixed-size run).
 */
#include <pthread.h>
#include <stdarg.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_SPARBIT = 0, ORACLE_RING = 1, ORACLE_RD = 2, ORACLE_BRUCK = 3, ORACLE_NE = 4 };
enum { SPACE_SEND = 0, SPACE_RECV = 1, SPACE_SCRATCH = 2 };

typedef struct {
    int32_t phase;     /* -1 own copy, 0..K-1 steps, K Bruck rotation */
    int32_t src_rank;
    int32_t dst_rank;
    int32_t src_space; /* SPACE_* */
    int32_t src_slot;  /* displacement in blocks inside src_rank's buffer of that space */
    int32_t dst_space;
    int32_t dst_slot;
} oracle_msg;

/* one posted MPI_Isend or MPI_Irecv: (peer, displacement in blocks, count = 1) at a step */
typedef struct {
    int32_t step;
    int32_t peer;
    int32_t space;
    int32_t slot;
} post_t;

typedef struct {
    post_t *v;
    size_t n, cap;
} postlist_t;

typedef struct {
    int algo;
    int P;
    int K;             /* number of communication steps */
    int has_rotation;  /* Bruck */
    oracle_msg *msgs;  /* ordered by phase */
    size_t n_msgs;
    size_t *phase_begin; /* index of first message of phase p at [p+1]; K+3 entries */
} oracle_plan;

static __thread char g_err[512];

static void set_err(const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
}

const char *oracle_last_error(void) { return g_err; }

static int post_push(postlist_t *l, int step, int peer, int space, int slot) {
    if (l->n == l->cap) {
        size_t nc = l->cap ? l->cap * 2 : 16;
        post_t *nv = (post_t *)realloc(l->v, nc * sizeof(post_t));
        if (!nv) return -1;
        l->v = nv;
        l->cap = nc;
    }
    l->v[l->n].step = step;
    l->v[l->n].peer = peer;
    l->v[l->n].space = space;
    l->v[l->n].slot = slot;
    l->n++;
    return 0;
}

/* true non-negative modulus */
static int64_t pmod(int64_t a, int64_t p) {
    int64_t r = a % p;
    return r < 0 ? r + p : r;
}

static int ceil_log2(unsigned p) {
    int k = 0;
    while ((1ull << k) < p) k++;
    return k;
}

static int floor_log2(unsigned p) {
    int k = 0;
    while ((2ull << k) <= p) k++;
    return k;
}

/* ---------------------------------------------------------------- Sparbit: Algorithm 1 ------ */
static int sparbit_rank_posts(int p, int rank, postlist_t *sends, postlist_t *recvs) {
    int K = ceil_log2((unsigned)p);
    if (K == 0) return 0; /* p = 1: the loop body never runs */
    uint32_t data = 1;
    uint32_t ignore = 0;
    uint32_t d = 1u << (K - 1);
    uint32_t last_ignore = (uint32_t)__builtin_ctz((unsigned)p);
    uint32_t ignore_steps = (~((uint32_t)p >> last_ignore) | 1u) << last_ignore;
    for (int i = 0; i < K; i++) {
        if (d & ignore_steps) ignore = 1;
        for (uint32_t j = 0; j < data - ignore; j++) {
            int64_t back_send = (int64_t)(2 * (uint64_t)j) * d;
            int64_t back_recv = (int64_t)(2 * (uint64_t)j + 1) * d;
            if (back_recv > p - 1) {
                set_err("sparbit: rank %d step %d j %u reaches back %lld >= p", rank, i, j,
                        (long long)back_recv);
                return -1;
            }
            if (post_push(sends, i, (int)pmod((int64_t)rank + d, p), SPACE_RECV,
                          (int)pmod((int64_t)rank - back_send, p)))
                return -1;
            if (post_push(recvs, i, (int)pmod((int64_t)rank - d, p), SPACE_RECV,
                          (int)pmod((int64_t)rank - back_recv, p)))
                return -1;
        }
        /* MPI_Waitall happens here: the simulator applies a step only after every rank posted */
        d >>= 1;
        data = (data << 1) - ignore;
        ignore = 0;
    }
    return 0;
}

/* ---------------------------------------------------------------- Ring ---------------------- */
static int ring_rank_posts(int p, int rank, postlist_t *sends, postlist_t *recvs) {
    int forward = rank; /* own block on the first step, then the block received last */
    for (int s = 0; s < p - 1; s++) {
        int arriving = (int)pmod((int64_t)rank - (s + 1), p); /* block of the rank s+1 behind */
        if (post_push(sends, s, (rank + 1) % p, SPACE_RECV, forward)) return -1;
        if (post_push(recvs, s, (int)pmod((int64_t)rank - 1, p), SPACE_RECV, arriving)) return -1;
        forward = arriving;
    }
    return 0;
}

/* ---------------------------------------------------------------- Recursive doubling -------- */
static int rd_rank_posts(int p, int rank, postlist_t *sends, postlist_t *recvs) {
    int K = ceil_log2((unsigned)p);
    for (int s = 0; s < K; s++) {
        int partner = rank ^ (1 << s);
        int held = 1 << s; /* everything received so far: the aligned group of 2^s ranks */
        int mine = (rank >> s) << s;
        int theirs = (partner >> s) << s;
        for (int j = 0; j < held; j++) {
            if (post_push(sends, s, partner, SPACE_RECV, mine + j)) return -1;
            if (post_push(recvs, s, partner, SPACE_RECV, theirs + j)) return -1;
        }
    }
    return 0;
}

/* ---------------------------------------------------------------- Neighbor exchange --------- */
static int ne_partner(int p, int rank, int s) {
    int sign = (s % 2 == 0) ? 1 : -1;                 /* (-1)^s */
    int to = (rank % 2 == 0) ? rank + sign : rank - sign;
    return (int)pmod(to, p);
}

/* first[s * p + x]: first of the (one or two) consecutive slots rank x sends on step s */
static int *ne_send_table(int p) {
    int steps = p / 2;
    int *first = (int *)malloc((size_t)(steps > 0 ? steps : 1) * (size_t)p * sizeof(int));
    if (!first) return NULL;
    for (int s = 0; s < steps; s++)
        for (int x = 0; x < p; x++) {
            if (s == 0)
                first[x] = x;                           /* the own block */
            else if (s == 1)
                first[p + x] = x - x % 2;               /* the two it holds: own and step 0's */
            else                                        /* what arrived on the previous step */
                first[s * p + x] = first[(s - 1) * p + ne_partner(p, x, s - 1)];
        }
    return first;
}

static int ne_rank_posts(int p, int rank, const int *first, postlist_t *sends, postlist_t *recvs) {
    for (int s = 0; s < p / 2; s++) {
        int partner = ne_partner(p, rank, s);
        int n = s == 0 ? 1 : 2;
        for (int j = 0; j < n; j++) {
            if (post_push(sends, s, partner, SPACE_RECV, first[s * p + rank] + j)) return -1;
            if (post_push(recvs, s, partner, SPACE_RECV, first[s * p + partner] + j)) return -1;
        }
    }
    return 0;
}

/* ---------------------------------------------------------------- Bruck --------------------- */
static int bruck_rank_posts(int p, int rank, postlist_t *sends, postlist_t *recvs) {
    int F = floor_log2((unsigned)p);
    int s;
    for (s = 0; s < F; s++) {
        int dist = 1 << s;
        for (int j = 0; j < dist; j++) { /* all the data it has: local slots [0, 2^s) */
            if (post_push(sends, s, (int)pmod((int64_t)rank - dist, p), SPACE_SCRATCH, j))
                return -1;
            if (post_push(recvs, s, (rank + dist) % p, SPACE_SCRATCH, dist + j)) return -1;
        }
    }
    if ((1 << F) != p) { /* additional step: only the first p - 2^floor(log2 p) blocks */
        int dist = 1 << F;
        int rest = p - dist;
        for (int j = 0; j < rest; j++) {
            if (post_push(sends, s, (int)pmod((int64_t)rank - dist, p), SPACE_SCRATCH, j))
                return -1;
            if (post_push(recvs, s, (rank + dist) % p, SPACE_SCRATCH, dist + j)) return -1;
        }
    }
    return 0;
}

/* ---------------------------------------------------------------- plan ---------------------- */
static void free_lists(postlist_t *l, int p) {
    if (!l) return;
    for (int r = 0; r < p; r++) free(l[r].v);
    free(l);
}

void oracle_plan_destroy(oracle_plan *pl) {
    if (!pl) return;
    free(pl->msgs);
    free(pl->phase_begin);
    free(pl);
}

static int msg_push(oracle_msg **v, size_t *n, size_t *cap, oracle_msg m) {
    if (*n == *cap) {
        size_t nc = *cap ? *cap * 2 : 64;
        oracle_msg *nv = (oracle_msg *)realloc(*v, nc * sizeof(oracle_msg));
        if (!nv) return -1;
        *v = nv;
        *cap = nc;
    }
    (*v)[(*n)++] = m;
    return 0;
}

/* Symbolic run of the message list: validity, single write, block identity.  ident[] holds the
 * rank whose block a location carries, or -1 when the location is not valid. */
static int check_plan(const oracle_plan *pl) {
    const int P = pl->P;
    const size_t PP = (size_t)P * P;
    int32_t *ident_recv = (int32_t *)malloc(PP * sizeof(int32_t));
    int32_t *ident_scr = (int32_t *)malloc(PP * sizeof(int32_t));
    int32_t *pend_recv = (int32_t *)malloc(PP * sizeof(int32_t)); /* written in this phase */
    int32_t *pend_scr = (int32_t *)malloc(PP * sizeof(int32_t));
    int32_t *writes_recv = (int32_t *)calloc(PP, sizeof(int32_t));
    int64_t *from_others = (int64_t *)calloc((size_t)P, sizeof(int64_t));
    int rc = -1;
    if (!ident_recv || !ident_scr || !pend_recv || !pend_scr || !writes_recv || !from_others) {
        set_err("out of memory in check_plan");
        goto done;
    }
    for (size_t i = 0; i < PP; i++) ident_recv[i] = ident_scr[i] = pend_recv[i] = pend_scr[i] = -1;

    for (int ph = -1; ph <= pl->K; ph++) {
        size_t b = pl->phase_begin[ph + 1], e = pl->phase_begin[ph + 2];
        for (size_t k = b; k < e; k++) {
            const oracle_msg *m = &pl->msgs[k];
            int32_t carried;
            if (m->src_rank < 0 || m->src_rank >= P || m->dst_rank < 0 || m->dst_rank >= P) {
                set_err("message %zu: rank out of range", k);
                goto done;
            }
            if (m->src_space == SPACE_SEND) {
                if (m->src_slot != 0) {
                    set_err("message %zu: send buffer has one slot", k);
                    goto done;
                }
                carried = m->src_rank;
            } else {
                if (m->src_slot < 0 || m->src_slot >= P) {
                    set_err("message %zu: source slot out of range", k);
                    goto done;
                }
                size_t at = (size_t)m->src_rank * P + m->src_slot;
                carried = (m->src_space == SPACE_RECV ? ident_recv : ident_scr)[at];
                if (carried < 0) {
                    set_err("phase %d: rank %d sends slot %d (space %d) it does not hold yet", ph,
                            m->src_rank, m->src_slot, m->src_space);
                    goto done;
                }
            }
            if (m->dst_space == SPACE_SEND || m->dst_slot < 0 || m->dst_slot >= P) {
                set_err("message %zu: bad destination", k);
                goto done;
            }
            size_t at = (size_t)m->dst_rank * P + m->dst_slot;
            int32_t *ident = m->dst_space == SPACE_RECV ? ident_recv : ident_scr;
            int32_t *pend = m->dst_space == SPACE_RECV ? pend_recv : pend_scr;
            if (ident[at] >= 0 || pend[at] >= 0) {
                set_err("phase %d: rank %d slot %d (space %d) written twice", ph, m->dst_rank,
                        m->dst_slot, m->dst_space);
                goto done;
            }
            pend[at] = carried;
            if (m->dst_space == SPACE_RECV) writes_recv[at]++;
            if (m->src_rank != m->dst_rank) from_others[m->dst_rank]++;
        }
        /* "Waitall": what arrived in this phase becomes valid for the next one */
        for (size_t k = b; k < e; k++) {
            const oracle_msg *m = &pl->msgs[k];
            size_t at = (size_t)m->dst_rank * P + m->dst_slot;
            if (m->dst_space == SPACE_RECV) {
                ident_recv[at] = pend_recv[at];
                pend_recv[at] = -1;
            } else {
                ident_scr[at] = pend_scr[at];
                pend_scr[at] = -1;
            }
        }
    }
    for (int r = 0; r < P; r++) {
        for (int b = 0; b < P; b++) {
            size_t at = (size_t)r * P + b;
            if (ident_recv[at] != b) {
                set_err("final state: rank %d slot %d carries block %d", r, b, ident_recv[at]);
                goto done;
            }
            if (writes_recv[at] != 1) {
                set_err("final state: rank %d slot %d written %d times", r, b, writes_recv[at]);
                goto done;
            }
        }
        if (from_others[r] != P - 1) {
            set_err("rank %d received %lld blocks from other ranks, expected %d", r,
                    (long long)from_others[r], P - 1);
            goto done;
        }
    }
    rc = 0;
done:
    free(ident_recv);
    free(ident_scr);
    free(pend_recv);
    free(pend_scr);
    free(writes_recv);
    free(from_others);
    return rc;
}

oracle_plan *oracle_plan_create(int algo, int P) {
    g_err[0] = 0;
    if (P < 1) {
        set_err("P must be >= 1");
        return NULL;
    }
    if (algo < ORACLE_SPARBIT || algo > ORACLE_NE) {
        set_err("unknown algorithm %d", algo);
        return NULL;
    }
    if (algo == ORACLE_RD && (P & (P - 1)) != 0) {
        set_err("recursive doubling is defined for powers of two only");
        return NULL;
    }
    if (algo == ORACLE_NE && P % 2 != 0) {
        set_err("neighbor exchange works with an even number of processes only");
        return NULL;
    }
    int *ne_first = NULL;
    oracle_plan *pl = (oracle_plan *)calloc(1, sizeof *pl);
    postlist_t *sends = (postlist_t *)calloc((size_t)P, sizeof(postlist_t));
    postlist_t *recvs = (postlist_t *)calloc((size_t)P, sizeof(postlist_t));
    size_t *cursor = (size_t *)calloc((size_t)P, sizeof(size_t));     /* per sender: next send */
    size_t *recv_cursor = (size_t *)calloc((size_t)P, sizeof(size_t)); /* per receiver */
    uint8_t **matched = (uint8_t **)calloc((size_t)P, sizeof(uint8_t *));
    size_t cap = 0;
    if (!pl || !sends || !recvs || !cursor || !recv_cursor || !matched) {
        set_err("out of memory");
        goto fail;
    }
    pl->algo = algo;
    pl->P = P;
    pl->K = algo == ORACLE_RING ? P - 1 : algo == ORACLE_NE ? P / 2 : ceil_log2((unsigned)P);
    if (algo == ORACLE_NE) {
        ne_first = ne_send_table(P);
        if (!ne_first) {
            set_err("out of memory");
            goto fail;
        }
    }
    pl->has_rotation = algo == ORACLE_BRUCK;

    /* every rank runs the algorithm on its own and posts its operations */
    for (int r = 0; r < P; r++) {
        int rc = 0;
        switch (algo) {
            case ORACLE_SPARBIT: rc = sparbit_rank_posts(P, r, &sends[r], &recvs[r]); break;
            case ORACLE_RING: rc = ring_rank_posts(P, r, &sends[r], &recvs[r]); break;
            case ORACLE_RD: rc = rd_rank_posts(P, r, &sends[r], &recvs[r]); break;
            case ORACLE_BRUCK: rc = bruck_rank_posts(P, r, &sends[r], &recvs[r]); break;
            case ORACLE_NE: rc = ne_rank_posts(P, r, ne_first, &sends[r], &recvs[r]); break;
        }
        if (rc) {
            if (!g_err[0]) set_err("out of memory while posting");
            goto fail;
        }
        matched[r] = (uint8_t *)calloc(sends[r].n ? sends[r].n : 1, 1);
        if (!matched[r]) {
            set_err("out of memory");
            goto fail;
        }
    }

    pl->phase_begin = (size_t *)calloc((size_t)pl->K + 3, sizeof(size_t));
    if (!pl->phase_begin) {
        set_err("out of memory");
        goto fail;
    }

    /* phase -1: own block into place */
    pl->phase_begin[0] = 0;
    for (int r = 0; r < P; r++) {
        oracle_msg m = {-1, r, r, SPACE_SEND, 0, algo == ORACLE_BRUCK ? SPACE_SCRATCH : SPACE_RECV,
                        algo == ORACLE_BRUCK ? 0 : r};
        if (msg_push(&pl->msgs, &pl->n_msgs, &cap, m)) {
            set_err("out of memory");
            goto fail;
        }
    }

    /* steps: match the k-th send a->b with the k-th receive b posted for a */
    for (int step = 0; step < pl->K; step++) {
        pl->phase_begin[step + 1] = pl->n_msgs;
        for (int dst = 0; dst < P; dst++) {
            postlist_t *rl = &recvs[dst];
            while (recv_cursor[dst] < rl->n && rl->v[recv_cursor[dst]].step == step) {
                post_t *rv = &rl->v[recv_cursor[dst]++];
                int src = rv->peer;
                postlist_t *sl = &sends[src];
                size_t k = cursor[src];
                while (k < sl->n && sl->v[k].step == step && (matched[src][k] || sl->v[k].peer != dst))
                    k++;
                if (k >= sl->n || sl->v[k].step != step) {
                    set_err("step %d: rank %d expects a block from %d that is never sent", step,
                            dst, src);
                    goto fail;
                }
                matched[src][k] = 1;
                while (cursor[src] < sl->n && matched[src][cursor[src]]) cursor[src]++;
                post_t *sv = &sl->v[k];
                if (algo != ORACLE_BRUCK && sv->slot != rv->slot) {
                    set_err("step %d: %d->%d displacement mismatch (%d vs %d)", step, src, dst,
                            sv->slot, rv->slot);
                    goto fail;
                }
                oracle_msg m = {step, src, dst, sv->space, sv->slot, rv->space, rv->slot};
                if (msg_push(&pl->msgs, &pl->n_msgs, &cap, m)) {
                    set_err("out of memory");
                    goto fail;
                }
            }
        }
        /* no send of this step may stay unmatched */
        for (int src = 0; src < P; src++) {
            postlist_t *sl = &sends[src];
            if (cursor[src] < sl->n && sl->v[cursor[src]].step == step) {
                set_err("step %d: rank %d sends a block to %d that is never received", step, src,
                        sl->v[cursor[src]].peer);
                goto fail;
            }
        }
    }
    for (int r = 0; r < P; r++) {
        if (cursor[r] != sends[r].n || recv_cursor[r] != recvs[r].n) {
            set_err("rank %d posted operations beyond the last step", r);
            goto fail;
        }
    }
    pl->phase_begin[pl->K + 1] = pl->n_msgs;

    /* Bruck's rotation: working slot i of rank r is the block of rank (r + i) mod P */
    if (pl->has_rotation) {
        for (int r = 0; r < P; r++)
            for (int i = 0; i < P; i++) {
                oracle_msg m = {pl->K, r, r, SPACE_SCRATCH, i, SPACE_RECV, (r + i) % P};
                if (msg_push(&pl->msgs, &pl->n_msgs, &cap, m)) {
                    set_err("out of memory");
                    goto fail;
                }
            }
    }
    pl->phase_begin[pl->K + 2] = pl->n_msgs;

    if (check_plan(pl)) goto fail;

    free(ne_first);
    free_lists(sends, P);
    free_lists(recvs, P);
    free(cursor);
    free(recv_cursor);
    for (int r = 0; r < P; r++) free(matched[r]);
    free(matched);
    return pl;
fail:
    free(ne_first);
    free_lists(sends, P);
    free_lists(recvs, P);
    free(cursor);
    free(recv_cursor);
    if (matched)
        for (int r = 0; r < P; r++) free(matched[r]);
    free(matched);
    oracle_plan_destroy(pl);
    return NULL;
}

int oracle_plan_num_steps(const oracle_plan *pl) { return pl ? pl->K : -1; }
int oracle_plan_has_rotation(const oracle_plan *pl) { return pl ? pl->has_rotation : -1; }
size_t oracle_plan_num_messages(const oracle_plan *pl) { return pl ? pl->n_msgs : 0; }
const oracle_msg *oracle_plan_messages(const oracle_plan *pl) { return pl ? pl->msgs : NULL; }

/* index range [*begin, *end) of the messages of one phase (-1 .. K) */
int oracle_plan_phase_range(const oracle_plan *pl, int phase, size_t *begin, size_t *end) {
    if (!pl || phase < -1 || phase > pl->K) return -1;
    *begin = pl->phase_begin[phase + 1];
    *end = pl->phase_begin[phase + 2];
    return 0;
}

/* ---------------------------------------------------------------- execution ----------------- */
typedef struct {
    const oracle_plan *pl;
    size_t m;
    const uint64_t *off; /* allgatherv: P+1 prefix sums of the blocks' byte counts, else NULL */
    const uint8_t *send;
    uint8_t *recv;
    uint8_t *scratch;
    int first, last;
    int tid, nthreads;
    pthread_barrier_t *bar;
} exec_arg;

static uint8_t *locate(const exec_arg *a, int space, int rank, int slot) {
    const size_t P = (size_t)a->pl->P;
    if (a->off) { /* block b is off[b+1]-off[b] bytes, at off[b] in the send buffer and in every
                     receive buffer (each receive buffer is off[P] bytes) */
        if (space == SPACE_SEND) return (uint8_t *)a->send + a->off[rank];
        return a->recv + (size_t)rank * a->off[P] + a->off[slot];
    }
    switch (space) {
        case SPACE_SEND: return (uint8_t *)a->send + (size_t)rank * a->m;
        case SPACE_RECV: return a->recv + ((size_t)rank * P + (size_t)slot) * a->m;
        default: return a->scratch + ((size_t)rank * P + (size_t)slot) * a->m;
    }
}

static void *exec_thread(void *vp) {
    exec_arg *a = (exec_arg *)vp;
    for (int ph = a->first; ph <= a->last; ph++) {
        size_t b = a->pl->phase_begin[ph + 1], e = a->pl->phase_begin[ph + 2];
        size_t n = e - b;
        size_t lo = b + n * (size_t)a->tid / (size_t)a->nthreads;
        size_t hi = b + n * ((size_t)a->tid + 1) / (size_t)a->nthreads;
        for (size_t k = lo; k < hi; k++) {
            const oracle_msg *m = &a->pl->msgs[k];
            /* the block a message carries is the one whose final slot it is written to */
            size_t bytes = a->off ? (size_t)(a->off[m->dst_slot + 1] - a->off[m->dst_slot]) : a->m;
            memcpy(locate(a, m->dst_space, m->dst_rank, m->dst_slot),
                   locate(a, m->src_space, m->src_rank, m->src_slot), bytes);
        }
        if (a->bar) pthread_barrier_wait(a->bar); /* the step's Waitall */
    }
    return NULL;
}

/*
 * Run phases first..last (inclusive, -1 .. K where K is only meaningful for Bruck) on host
 * buffers.  send: P*m bytes.  recv: P*P*m bytes.  scratch: P*P*m bytes, Bruck only (else may be
 * NULL).  Buffers are not initialised here: the caller fills recv/scratch with its sentinel.
 * threads >= 1; messages of a phase are split evenly between threads (their writes are disjoint,
 * which check_plan proved), with a barrier after every phase.
 */
static int run_impl(const oracle_plan *pl, size_t m, const uint64_t *off, const void *send, void *recv,
                    void *scratch, int first, int last, int threads);

int oracle_run(const oracle_plan *pl, size_t m, const void *send, void *recv, void *scratch,
               int first, int last, int threads) {
    return run_impl(pl, m, NULL, send, recv, scratch, first, last, threads);
}

/*
 * The same phases for blocks of different sizes (MPI_Allgatherv with contiguous displacements;
 * the paper's conclusion names it as the next target, and the schedules never look inside a
 * block).  off: P+1 prefix sums of the byte counts.  send: off[P] bytes, rank r's block at off[r].
 * recv: P * off[P] bytes, rank r's buffer at r * off[P], block j at + off[j].  Not for Bruck (its
 * rotated working buffer is laid out for equal blocks).
 */
int oracle_run_v(const oracle_plan *pl, const uint64_t *off, const void *send, void *recv, int first,
                 int last, int threads) {
    if (!pl || !off) {
        set_err("null argument");
        return -1;
    }
    if (pl->algo == ORACLE_BRUCK) {
        set_err("Bruck is laid out for equal blocks");
        return -1;
    }
    return run_impl(pl, off[pl->P] ? 1 : 0, off, send, recv, NULL, first, last, threads);
}

static int run_impl(const oracle_plan *pl, size_t m, const uint64_t *off, const void *send, void *recv,
                    void *scratch, int first, int last, int threads) {
    if (!pl) {
        set_err("null plan");
        return -1;
    }
    int max_phase = pl->has_rotation ? pl->K : pl->K - 1;
    if (first < -1) first = -1;
    if (last > max_phase) last = max_phase;
    if (first > last || m == 0) return 0;
    if (!send || !recv || (pl->algo == ORACLE_BRUCK && !scratch)) {
        set_err("null buffer");
        return -1;
    }
    if (threads < 1) threads = 1;
    if (threads == 1) {
        exec_arg a = {pl, m, off, (const uint8_t *)send, (uint8_t *)recv, (uint8_t *)scratch,
                      first, last, 0, 1, NULL};
        exec_thread(&a);
        return 0;
    }
    pthread_barrier_t bar;
    pthread_barrier_init(&bar, NULL, (unsigned)threads);
    pthread_t *th = (pthread_t *)malloc((size_t)threads * sizeof(pthread_t));
    exec_arg *args = (exec_arg *)malloc((size_t)threads * sizeof(exec_arg));
    if (!th || !args) {
        free(th);
        free(args);
        set_err("out of memory");
        return -1;
    }
    for (int t = 0; t < threads; t++) {
        exec_arg a = {pl, m, off, (const uint8_t *)send, (uint8_t *)recv, (uint8_t *)scratch,
                      first, last, t, threads, &bar};
        args[t] = a;
        pthread_create(&th[t], NULL, exec_thread, &args[t]);
    }
    for (int t = 0; t < threads; t++) pthread_join(th[t], NULL);
    pthread_barrier_destroy(&bar);
    free(th);
    free(args);
    return 0;
}
