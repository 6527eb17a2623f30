/*
 * ORACLE (test infrastructure, not the product): chess rules, legal-move masks,
 * policy index maps and the input-plane encoder, written plainly for the CPU.
 *
 * Nothing here is shared with the CUDA library or with the input generator.
 * Board: 10x12 mailbox with an off-board border, so that stepping off the board
 * is detected by a sentinel rather than by coordinate tests.
 *
 * What each part follows:
 *  - leaf evaluation takes a batch of independent positions and returns priors
 *    over legal moves plus a value for the player to move (Sec. 3.1, Sec. 3.6);
 *  - planes are side-to-move canonical: for Black to move ranks are reflected and
 *    colours exchanged, files keep their order; row 0 is the mover's home rank,
 *    column 0 is file a; flags and scalars fill all 64 squares (App. D.1, Table D.1);
 *  - own pieces P,N,B,R,Q,K come before the opponent's, castling planes are ordered
 *    own king side, own queen side, opponent king side, opponent queen side, the
 *    halfmove clock is capped at 100, missing history is zero-filled (Table D.1);
 *  - in the action encoding castling is the king-to-own-rook pair and en passant
 *    is the pawn's ordinary origin-destination pair; the flat list has 1,792
 *    ray-or-knight pairs followed by promotion actions (App. D.1);
 *  - illegal actions are masked before the softmax over legal moves (App. D.1).
 * The 19- and 112-plane layouts, the 73-plane head and the three-piece promotion
 * list are the workload definitions' (see the encoder and index functions below).
 *
 * Pins (tests, CPU only): perft from the start position 20 / 400 / 8,902 / 197,281,
 * published perft counts of positions rich in castling, en passant and promotion,
 * move-set equality with the input generator's separate rules code, index-map
 * counts 1,792 / 22 / 1,858 / 4,672, plane invariants.
 */
#include <stdint.h>
#include <string.h>

enum { EMPTY = 0, OFF = 99 };
/* pieces 1..6 white P N B R Q K, 7..12 black P N B R Q K */

typedef struct {
    uint8_t sq[120];
    int stm;       /* 0 white, 1 black */
    int castling;  /* bit0 WK, bit1 WQ, bit2 BK, bit3 BQ */
    int ep;        /* mailbox index of the en-passant target square, 0 if none */
} MBoard;

typedef struct { int from, to, promo, flag; } MMove;
/* promo: 0 none, 1 N, 2 B, 3 R, 4 Q.  flag: 0 plain, 1 double push, 2 en passant, 3 O-O, 4 O-O-O.
 * from/to are 0..63 squares (file + 8*rank); for castling `to` is the king's destination. */

typedef struct {
    uint64_t pieces[12];
    uint8_t stm, castling, ep_square, halfmove, repetitions, pad[3];
} PosRecord;                      /* 104 bytes */
typedef struct {
    PosRecord cur;
    uint64_t hist_pieces[7][12];
    uint8_t hist_rep[7];
    uint8_t n_hist;
} PosRecordH8;                    /* 784 bytes */

static inline int mb(int s) { return 21 + (s & 7) + 10 * (s >> 3); }
static inline int sq64(int m) { return (m % 10 - 1) + 8 * (m / 10 - 2); }
static inline int colour(int p) { return p >= 7; }   /* valid for p in 1..12 */

static void load_record(const PosRecord *r, MBoard *b) {
    for (int i = 0; i < 120; ++i) b->sq[i] = OFF;
    for (int s = 0; s < 64; ++s) b->sq[mb(s)] = EMPTY;
    for (int p = 0; p < 12; ++p)
        for (int s = 0; s < 64; ++s)
            if ((r->pieces[p] >> s) & 1ULL) b->sq[mb(s)] = (uint8_t)(p + 1);
    b->stm = r->stm;
    b->castling = r->castling;
    b->ep = r->ep_square < 64 ? mb(r->ep_square) : 0;
}

static const int N_OFF[8] = { -21, -19, -12, -8, 8, 12, 19, 21 };
static const int K_OFF[8] = { -11, -10, -9, -1, 1, 9, 10, 11 };
static const int B_OFF[4] = { -11, -9, 9, 11 };
static const int R_OFF[4] = { -10, -1, 1, 10 };

/* is mailbox square m attacked by side `by`? */
static int is_attacked(const MBoard *b, int m, int by) {
    int base = by ? 6 : 0;
    int pawn = base + 1, knight = base + 2, bishop = base + 3, rook = base + 4, queen = base + 5, king = base + 6;
    /* a white pawn attacks the two squares diagonally ahead (+9, +11) of itself */
    if (by == 0) { if (b->sq[m - 9] == pawn || b->sq[m - 11] == pawn) return 1; }
    else         { if (b->sq[m + 9] == pawn || b->sq[m + 11] == pawn) return 1; }
    for (int i = 0; i < 8; ++i) {
        if (b->sq[m + N_OFF[i]] == knight) return 1;
        if (b->sq[m + K_OFF[i]] == king) return 1;
    }
    for (int i = 0; i < 4; ++i) {
        int t = m + B_OFF[i];
        while (b->sq[t] == EMPTY) t += B_OFF[i];
        if (b->sq[t] == bishop || b->sq[t] == queen) return 1;
        t = m + R_OFF[i];
        while (b->sq[t] == EMPTY) t += R_OFF[i];
        if (b->sq[t] == rook || b->sq[t] == queen) return 1;
    }
    return 0;
}

static int find_king(const MBoard *b, int side) {
    int k = side ? 12 : 6;
    for (int m = 21; m <= 98; ++m) if (b->sq[m] == k) return m;
    return 0;
}

static void play(MBoard *b, const MMove *mv) {
    int from = mb(mv->from), to = mb(mv->to);
    int p = b->sq[from], us = b->stm;
    b->sq[from] = EMPTY;
    b->sq[to] = (uint8_t)p;
    if (mv->flag == 2) b->sq[to + (us ? 10 : -10)] = EMPTY;
    if (mv->flag == 3) { b->sq[to + 1] = EMPTY; b->sq[to - 1] = (uint8_t)(us ? 10 : 4); }
    if (mv->flag == 4) { b->sq[to - 2] = EMPTY; b->sq[to + 1] = (uint8_t)(us ? 10 : 4); }
    if (mv->promo) b->sq[to] = (uint8_t)((us ? 6 : 0) + 1 + mv->promo);
    if (p == 6) b->castling &= ~3;
    if (p == 12) b->castling &= ~12;
    if (mv->from == 7 || mv->to == 7) b->castling &= ~1;
    if (mv->from == 0 || mv->to == 0) b->castling &= ~2;
    if (mv->from == 63 || mv->to == 63) b->castling &= ~4;
    if (mv->from == 56 || mv->to == 56) b->castling &= ~8;
    b->ep = (mv->flag == 1) ? (from + to) / 2 : 0;
    b->stm ^= 1;
}

static int push(MMove *list, int n, int from_m, int to_m, int promo, int flag) {
    list[n].from = sq64(from_m); list[n].to = sq64(to_m); list[n].promo = promo; list[n].flag = flag;
    return n + 1;
}

static int gen_pseudo(const MBoard *b, MMove *list) {
    int n = 0, us = b->stm, them = us ^ 1;
    for (int m = 21; m <= 98; ++m) {
        int p = b->sq[m];
        if (p == EMPTY || p == OFF || colour(p) != us) continue;
        int kind = us ? p - 6 : p;
        if (kind == 1) {
            int step = us ? -10 : 10;
            int home_row = us ? 8 : 3;     /* mailbox row index (m / 10) of the pawn's start rank */
            int last_row = us ? 2 : 9;     /* row of the promotion rank */
            int t = m + step;
            if (b->sq[t] == EMPTY) {
                if (t / 10 == last_row) for (int q = 1; q <= 4; ++q) n = push(list, n, m, t, q, 0);
                else {
                    n = push(list, n, m, t, 0, 0);
                    if (m / 10 == home_row && b->sq[t + step] == EMPTY) n = push(list, n, m, t + step, 0, 1);
                }
            }
            for (int side = -1; side <= 1; side += 2) {
                int c = t + side, q = b->sq[c];
                if (q == OFF) continue;
                if (q != EMPTY && colour(q) == them) {
                    if (c / 10 == last_row) for (int k = 1; k <= 4; ++k) n = push(list, n, m, c, k, 0);
                    else n = push(list, n, m, c, 0, 0);
                } else if (q == EMPTY && b->ep != 0 && c == b->ep) {
                    n = push(list, n, m, c, 0, 2);
                }
            }
        } else if (kind == 2 || kind == 6) {
            const int *off = (kind == 2) ? N_OFF : K_OFF;
            for (int i = 0; i < 8; ++i) {
                int t = m + off[i], q = b->sq[t];
                if (q == OFF) continue;
                if (q == EMPTY || colour(q) == them) n = push(list, n, m, t, 0, 0);
            }
            if (kind == 6) {
                int e = us ? 95 : 25;                    /* e8 / e1 */
                int rook = us ? 10 : 4;
                int kbit = us ? 4 : 1, qbit = us ? 8 : 2;
                if (m == e && !is_attacked(b, e, them)) {
                    if ((b->castling & kbit) && b->sq[e + 3] == rook && b->sq[e + 1] == EMPTY &&
                        b->sq[e + 2] == EMPTY && !is_attacked(b, e + 1, them) && !is_attacked(b, e + 2, them))
                        n = push(list, n, m, e + 2, 0, 3);
                    if ((b->castling & qbit) && b->sq[e - 4] == rook && b->sq[e - 1] == EMPTY &&
                        b->sq[e - 2] == EMPTY && b->sq[e - 3] == EMPTY &&
                        !is_attacked(b, e - 1, them) && !is_attacked(b, e - 2, them))
                        n = push(list, n, m, e - 2, 0, 4);
                }
            }
        } else {
            for (int i = 0; i < 4; ++i) {
                if (kind != 4) {   /* bishop or queen: diagonals */
                    int t = m + B_OFF[i];
                    while (b->sq[t] == EMPTY) { n = push(list, n, m, t, 0, 0); t += B_OFF[i]; }
                    if (b->sq[t] != OFF && colour(b->sq[t]) == them) n = push(list, n, m, t, 0, 0);
                }
                if (kind != 3) {   /* rook or queen: files and ranks */
                    int t = m + R_OFF[i];
                    while (b->sq[t] == EMPTY) { n = push(list, n, m, t, 0, 0); t += R_OFF[i]; }
                    if (b->sq[t] != OFF && colour(b->sq[t]) == them) n = push(list, n, m, t, 0, 0);
                }
            }
        }
    }
    return n;
}

static int gen_legal(const MBoard *b, MMove *out) {
    MMove tmp[256];
    int n = gen_pseudo(b, tmp), k = 0;
    for (int i = 0; i < n; ++i) {
        MBoard c = *b;
        play(&c, &tmp[i]);
        if (!is_attacked(&c, find_king(&c, b->stm), b->stm ^ 1)) out[k++] = tmp[i];
    }
    return k;
}

static uint64_t perft_rec(const MBoard *b, int depth) {
    MMove list[256];
    int n = gen_legal(b, list);
    if (depth == 1) return (uint64_t)n;
    uint64_t total = 0;
    for (int i = 0; i < n; ++i) {
        MBoard c = *b;
        play(&c, &list[i]);
        total += perft_rec(&c, depth - 1);
    }
    return total;
}

/* Number of leaf nodes of the legal-move tree of the given depth (>= 1). */
uint64_t orc_perft(const void *record, int depth) {
    MBoard b; load_record((const PosRecord *)record, &b);
    if (depth < 1) return 1;
    return perft_rec(&b, depth);
}

/* Legal moves as (from, to, promo) triples in generation order; castling reported as the
 * king's own move.  Returns the count (<= 256). */
int orc_legal_moves(const void *record, uint8_t *triples) {
    MBoard b; load_record((const PosRecord *)record, &b);
    MMove list[256];
    int n = gen_legal(&b, list);
    for (int i = 0; i < n; ++i) {
        triples[3 * i] = (uint8_t)list[i].from; triples[3 * i + 1] = (uint8_t)list[i].to;
        triples[3 * i + 2] = (uint8_t)list[i].promo;
    }
    return n;
}

/* ---- policy index maps (mover-oriented coordinates) ------------------------ */

/* 73-plane head: index = plane * 64 + origin.  Planes 0..55: direction
 * (N, NE, E, SE, S, SW, W, NW) x distance 1..7 -> 7*direction + distance-1;
 * 56..63: knight jumps (1,2),(2,1),(2,-1),(1,-2),(-1,-2),(-2,-1),(-2,1),(-1,2) as (file, rank) steps;
 * 64..72: promotion to N, B, R x (capture towards file-1, straight, capture towards file+1)
 * -> 64 + 3*piece + direction.  Queen promotions use the ordinary one-step plane. */
static int index73(int from, int to, int promo) {
    int df = (to & 7) - (from & 7), dr = (to >> 3) - (from >> 3);
    int plane;
    if (promo >= 1 && promo <= 3) {
        plane = 64 + 3 * (promo - 1) + (df + 1);
    } else {
        int adf = df < 0 ? -df : df, adr = dr < 0 ? -dr : dr;
        if ((adf == 1 && adr == 2) || (adf == 2 && adr == 1)) {
            static const int jf[8] = { 1, 2, 2, 1, -1, -2, -2, -1 };
            static const int jr[8] = { 2, 1, -1, -2, -2, -1, 1, 2 };
            plane = -1;
            for (int k = 0; k < 8; ++k) if (jf[k] == df && jr[k] == dr) plane = 56 + k;
        } else {
            int sf = (df > 0) - (df < 0), sr = (dr > 0) - (dr < 0);
            static const int dirf[8] = { 0, 1, 1, 1, 0, -1, -1, -1 };
            static const int dirr[8] = { 1, 1, 0, -1, -1, -1, 0, 1 };
            int d = -1;
            for (int k = 0; k < 8; ++k) if (dirf[k] == sf && dirr[k] == sr) d = k;
            int dist = adf > adr ? adf : adr;
            if (d < 0 || (adf != 0 && adr != 0 && adf != adr)) return -1;
            plane = 7 * d + dist - 1;
        }
    }
    return plane * 64 + from;
}

/* Flat list: all (origin, destination) with origin ascending then destination ascending that lie
 * a queen ray or a knight jump apart (1,792 of them), then for origins on the seventh rank the
 * destinations origin+7, +8, +9 that stay on the board, each with pieces N, B, R (22 x 3 = 66).
 * A pawn reaching the last rank through a plain pair promotes to a queen. */
static int16_t flat_pair[64][64];
static int16_t flat_promo[8][3];      /* [origin file][file step + 1] -> first of three indices */
static int flat_ready = 0;
static int flat_count = 0;
static void build_flat(void) {
    int n = 0;
    for (int f = 0; f < 64; ++f)
        for (int t = 0; t < 64; ++t) {
            flat_pair[f][t] = -1;
            if (f == t) continue;
            int df = (t & 7) - (f & 7), dr = (t >> 3) - (f >> 3);
            int adf = df < 0 ? -df : df, adr = dr < 0 ? -dr : dr;
            int ray = (df == 0 || dr == 0 || adf == adr);
            int jump = (adf == 1 && adr == 2) || (adf == 2 && adr == 1);
            if (ray || jump) flat_pair[f][t] = (int16_t)n++;
        }
    for (int file = 0; file < 8; ++file)
        for (int step = -1; step <= 1; ++step) {
            flat_promo[file][step + 1] = -1;
            if (file + step < 0 || file + step > 7) continue;
            flat_promo[file][step + 1] = (int16_t)n;
            n += 3;
        }
    flat_count = n;
    flat_ready = 1;
}
static int index_flat(int from, int to, int promo) {
    if (!flat_ready) build_flat();
    if (promo >= 1 && promo <= 3) {
        int base = flat_promo[from & 7][(to & 7) - (from & 7) + 1];
        return base < 0 ? -1 : base + (promo - 1);
    }
    return flat_pair[from][to];
}

int orc_flat_count(void) { if (!flat_ready) build_flat(); return flat_count; }

/* The paper's own action list (Sec. 3.2, App. D.1): the same 1,792 origin-destination pairs, in
 * the same order, then 88 explicit promotions: origins on the seventh rank ascending, destinations
 * origin+7, +8, +9 that stay on the board ascending, pieces in the order queen, rook, bishop,
 * knight (22 x 4).  A promoting pawn move has ONLY its promotion action; the plain pair of the
 * same two squares belongs to the other pieces that can make that step. */
static int index_fromto(int from, int to, int promo) {
    if (!flat_ready) build_flat();
    if (promo >= 1 && promo <= 4) {
        int step = (to & 7) - (from & 7);
        if ((from >> 3) != 6 || (to >> 3) != 7 || step < -1 || step > 1) return -1;
        int slot = 0;                       /* how many (file, step) combinations come before this one */
        for (int file = 0; file < 8; ++file)
            for (int st = -1; st <= 1; ++st) {
                if (file + st < 0 || file + st > 7) continue;
                if (file == (from & 7) && st == step) return 1792 + 4 * slot + (4 - promo);
                ++slot;
            }
        return -1;
    }
    return flat_pair[from][to];
}

/* Policy index of a move given in ABSOLUTE squares for the side `stm`; `castle` 0 none,
 * 1 short, 2 long.  Returns -1 if the move has no index. */
int orc_policy_index(int head, int stm, int from, int to, int promo, int castle) {
    if (castle) to = (stm ? 56 : 0) + (castle == 1 ? 7 : 0);   /* king takes the own-rook square */
    if (stm) { from ^= 56; to ^= 56; }                          /* reflect ranks for Black */
    return head == 0 ? index73(from, to, promo) : head == 1 ? index_flat(from, to, promo) : index_fromto(from, to, promo);
}

/* Legal-move masks: bit (i & 63) of word (i >> 6) is set iff policy index i is a legal move.
 * words = 73 (head 0) or 30 (head 1: 1,858 moves; head 2: the paper's 1,880 actions) per position.
 * Returns 0, or -1 if a move had no index. */
int orc_legal_masks(const void *records, int stride, int n, int head, uint64_t *masks) {
    int words = head == 0 ? 73 : 30, bad = 0;
    for (int i = 0; i < n; ++i) {
        const PosRecord *r = (const PosRecord *)((const char *)records + (size_t)i * stride);
        uint64_t *row = masks + (size_t)i * words;
        memset(row, 0, sizeof(uint64_t) * words);
        MBoard b; load_record(r, &b);
        MMove list[256];
        int k = gen_legal(&b, list);
        for (int j = 0; j < k; ++j) {
            int castle = list[j].flag == 3 ? 1 : list[j].flag == 4 ? 2 : 0;
            int idx = orc_policy_index(head, b.stm, list[j].from, list[j].to, list[j].promo, castle);
            if (idx < 0) { bad = 1; continue; }
            row[idx >> 6] |= 1ULL << (idx & 63);
        }
    }
    return bad ? -1 : 0;
}

/* ---- input planes ---------------------------------------------------------- */

static void put_board(double *planes, int first_plane, const uint64_t pieces[12], int stm) {
    /* planes first_plane..+5 own P..K, +6..+11 opponent P..K, in mover-oriented coordinates */
    for (int k = 0; k < 6; ++k) {
        uint64_t own = pieces[(stm ? 6 : 0) + k], opp = pieces[(stm ? 0 : 6) + k];
        for (int s = 0; s < 64; ++s) {
            int c = stm ? (s ^ 56) : s;
            if ((own >> s) & 1ULL) planes[(first_plane + k) * 64 + c] = 1.0;
            if ((opp >> s) & 1ULL) planes[(first_plane + 6 + k) * 64 + c] = 1.0;
        }
    }
}
static void fill(double *planes, int plane, double v) {
    for (int s = 0; s < 64; ++s) planes[plane * 64 + s] = v;
}
static double halfmove_value(int hm) {
    /* the clock is capped at 100 and divided by 100 in single precision, the arithmetic in which
     * the stored plane value is decided */
    float v = (float)(hm > 100 ? 100 : hm) / 100.0f;
    return (double)v;
}

/* planes_out: [n][in_planes][64] doubles, square index = row*8 + column in mover orientation.
 * in_planes 19: 0-5 own P..K, 6-11 opponent P..K, 12 one iff Black to move, 13-16 castling
 *   (own K-side, own Q-side, opponent K-side, opponent Q-side), 17 min(halfmove,100)/100,
 *   18 one iff the position occurred earlier in its game.
 * in_planes 112: for t = 0..7, planes 13t..13t+11 the board t plies ago (own then opponent, all
 *   oriented by the CURRENT mover), 13t+12 that board's repetition flag, zero where the game is
 *   shorter; 104-107 castling as above, 108 one iff Black to move, 109 halfmove/100, 110 zeros,
 *   111 ones.  (records must then be 784-byte records with history.) */
int orc_encode(const void *records, int stride, int n, int in_planes, double *planes_out) {
    if (in_planes != 19 && in_planes != 112) return -1;
    for (int i = 0; i < n; ++i) {
        const PosRecord *r = (const PosRecord *)((const char *)records + (size_t)i * stride);
        double *pl = planes_out + (size_t)i * in_planes * 64;
        memset(pl, 0, sizeof(double) * in_planes * 64);
        int stm = r->stm;
        int ownK = stm ? 4 : 1, ownQ = stm ? 8 : 2, oppK = stm ? 1 : 4, oppQ = stm ? 2 : 8;
        if (in_planes == 19) {
            put_board(pl, 0, r->pieces, stm);
            if (stm) fill(pl, 12, 1.0);
            if (r->castling & ownK) fill(pl, 13, 1.0);
            if (r->castling & ownQ) fill(pl, 14, 1.0);
            if (r->castling & oppK) fill(pl, 15, 1.0);
            if (r->castling & oppQ) fill(pl, 16, 1.0);
            fill(pl, 17, halfmove_value(r->halfmove));
            if (r->repetitions >= 1) fill(pl, 18, 1.0);
        } else {
            const PosRecordH8 *h = (const PosRecordH8 *)r;
            put_board(pl, 0, r->pieces, stm);
            if (r->repetitions >= 1) fill(pl, 12, 1.0);
            for (int t = 1; t <= 7 && t <= h->n_hist; ++t) {
                put_board(pl, 13 * t, h->hist_pieces[t - 1], stm);
                if (h->hist_rep[t - 1] >= 1) fill(pl, 13 * t + 12, 1.0);
            }
            if (r->castling & ownK) fill(pl, 104, 1.0);
            if (r->castling & ownQ) fill(pl, 105, 1.0);
            if (r->castling & oppK) fill(pl, 106, 1.0);
            if (r->castling & oppQ) fill(pl, 107, 1.0);
            if (stm) fill(pl, 108, 1.0);
            fill(pl, 109, halfmove_value(r->halfmove));
            fill(pl, 111, 1.0);
        }
    }
    return 0;
}

/* ---- the 52 input planes of the paper's network (App. D.1, Table D.1) -----------------------
 * records: 128-byte records = the 104-byte position, then move_from[8], move_to[8] (absolute
 * squares, most recent move first, castling as the king's own move), n_moves, padding.
 * planes_out: [n][52][64] doubles in mover orientation (Black to move: ranks reflected, colours
 * exchanged, files kept; row 0 = the mover's home rank, column 0 = file a).
 *   0-5 own P N B R Q K, 6-11 opponent's; 12-15 castling rights own K-side, own Q-side, opponent
 *   K-side, opponent Q-side; 16 all own pieces, 17 all opponent pieces; 18 the opponent pieces
 *   that give check; 19 the en-passant target square; 20 / 21 one iff the position occurred at
 *   least once / twice before; 22+2t, 23+2t origin and destination of the move t plies back
 *   (t = 0..7, zero where the game is shorter); 38 checkerboard fixed in these coordinates, the
 *   a1 corner (row 0, column 0) set; 39 one iff each side has exactly one bishop and the two stand
 *   on squares of different colour; 40-45 own minus opponent count of P N B R Q K; 46 halfmove
 *   clock capped at 100, as a count; 47-51 own count of P N B R Q.
 * Readings where the table is silent: plane 19 is set whenever the record carries an en-passant
 * square (the square behind a pawn that has just advanced two ranks), whether or not a capture
 * there is legal; counts and the clock are plain integers, not normalised. */
typedef struct {
    PosRecord cur;
    uint8_t move_from[8], move_to[8];
    uint8_t n_moves;
    uint8_t pad[7];
} PosRecordM8;                    /* 128 bytes */

static int popcount64(uint64_t v) { int n = 0; while (v) { v &= v - 1; ++n; } return n; }

int orc_encode52(const void *records, int stride, int n, double *planes_out) {
    for (int i = 0; i < n; ++i) {
        const PosRecordM8 *m8 = (const PosRecordM8 *)((const char *)records + (size_t)i * stride);
        const PosRecord *r = &m8->cur;
        double *pl = planes_out + (size_t)i * 52 * 64;
        memset(pl, 0, sizeof(double) * 52 * 64);
        const int stm = r->stm;
        const int flip = stm ? 56 : 0;
        const int ownK = stm ? 4 : 1, ownQ = stm ? 8 : 2, oppK = stm ? 1 : 4, oppQ = stm ? 2 : 8;
        put_board(pl, 0, r->pieces, stm);
        if (r->castling & ownK) fill(pl, 12, 1.0);
        if (r->castling & ownQ) fill(pl, 13, 1.0);
        if (r->castling & oppK) fill(pl, 14, 1.0);
        if (r->castling & oppQ) fill(pl, 15, 1.0);
        for (int k = 0; k < 6; ++k)
            for (int s = 0; s < 64; ++s) {
                if (pl[k * 64 + s] != 0.0) pl[16 * 64 + s] = 1.0;
                if (pl[(6 + k) * 64 + s] != 0.0) pl[17 * 64 + s] = 1.0;
            }
        /* checkers: walk from the mover's king outwards and see which enemy piece looks back */
        {
            MBoard b; load_record(r, &b);
            const int km = find_king(&b, stm);
            const int eb = stm ? 0 : 6;        /* enemy piece codes eb+1 .. eb+6 */
            if (km) {
                /* an enemy pawn checks from the two squares diagonally in front of the king (seen from the mover) */
                const int fwd = stm ? -10 : 10;
                for (int d = -1; d <= 1; d += 2)
                    if (b.sq[km + fwd + d] == eb + 1) pl[18 * 64 + (sq64(km + fwd + d) ^ flip)] = 1.0;
                for (int j = 0; j < 8; ++j)
                    if (b.sq[km + N_OFF[j]] == eb + 2) pl[18 * 64 + (sq64(km + N_OFF[j]) ^ flip)] = 1.0;
                for (int j = 0; j < 4; ++j) {
                    int t = km + B_OFF[j];
                    while (b.sq[t] == EMPTY) t += B_OFF[j];
                    if (b.sq[t] == eb + 3 || b.sq[t] == eb + 5) pl[18 * 64 + (sq64(t) ^ flip)] = 1.0;
                    t = km + R_OFF[j];
                    while (b.sq[t] == EMPTY) t += R_OFF[j];
                    if (b.sq[t] == eb + 4 || b.sq[t] == eb + 5) pl[18 * 64 + (sq64(t) ^ flip)] = 1.0;
                }
            }
        }
        if (r->ep_square < 64) pl[19 * 64 + (r->ep_square ^ flip)] = 1.0;
        if (r->repetitions >= 1) fill(pl, 20, 1.0);
        if (r->repetitions >= 2) fill(pl, 21, 1.0);
        for (int t = 0; t < 8 && t < m8->n_moves; ++t) {
            pl[(22 + 2 * t) * 64 + (m8->move_from[t] ^ flip)] = 1.0;
            pl[(23 + 2 * t) * 64 + (m8->move_to[t] ^ flip)] = 1.0;
        }
        for (int row = 0; row < 8; ++row)
            for (int col = 0; col < 8; ++col)
                if (((row + col) & 1) == 0) pl[38 * 64 + row * 8 + col] = 1.0;
        int own_n[6], opp_n[6];
        for (int k = 0; k < 6; ++k) {
            own_n[k] = popcount64(r->pieces[(stm ? 6 : 0) + k]);
            opp_n[k] = popcount64(r->pieces[(stm ? 0 : 6) + k]);
        }
        if (own_n[2] == 1 && opp_n[2] == 1) {
            int a = 0, c = 0;
            for (int s = 0; s < 64; ++s) {
                if ((r->pieces[(stm ? 6 : 0) + 2] >> s) & 1ULL) a = ((s & 7) + (s >> 3)) & 1;
                if ((r->pieces[(stm ? 0 : 6) + 2] >> s) & 1ULL) c = ((s & 7) + (s >> 3)) & 1;
            }
            if (a != c) fill(pl, 39, 1.0);
        }
        for (int k = 0; k < 6; ++k) fill(pl, 40 + k, (double)(own_n[k] - opp_n[k]));
        fill(pl, 46, (double)(r->halfmove > 100 ? 100 : r->halfmove));
        for (int k = 0; k < 5; ++k) fill(pl, 47 + k, (double)own_n[k]);
    }
    return 0;
}

/* ---- applying an action to a position (the step a search tree takes from a node to its child) ----
 * actions[i] is a policy index of `head` (0: 73 planes, 1: 1,858 list, 2: 1,880 list) that is legal
 * in records[i]; out[i] receives the successor in the same record layout (stride 104, 784 or 128):
 * bitboards, side to move, castling rights (lost when the king or a rook leaves its home square or a
 * rook is captured there), en-passant square (set behind a pawn that advanced two ranks, else 64),
 * halfmove clock (0 after a pawn move or a capture, else one more, saturating at 255), repetitions 0
 * (a successor built this way does not know its game's earlier positions).  Records with history
 * get the old position pushed onto their seven boards, records with moves the move pushed onto
 * their eight (castling as the king's own move).  In the 73-plane and 1,858 lists a pawn that
 * reaches the last rank through a plain action becomes a queen.  Returns 0, or -1 if an action is
 * not a legal move of its position. */
int orc_apply_moves(const void *records, int stride, int n, int head, const int32_t *actions, void *out) {
    for (int i = 0; i < n; ++i) {
        const PosRecord *r = (const PosRecord *)((const char *)records + (size_t)i * stride);
        char *dst = (char *)out + (size_t)i * stride;
        MBoard b; load_record(r, &b);
        MMove list[256];
        int k = gen_legal(&b, list), found = -1;
        for (int j = 0; j < k && found < 0; ++j) {
            int castle = list[j].flag == 3 ? 1 : list[j].flag == 4 ? 2 : 0;
            if (orc_policy_index(head, b.stm, list[j].from, list[j].to, list[j].promo, castle) == actions[i]) found = j;
        }
        if (found < 0) return -1;
        const MMove mv = list[found];
        const int piece = b.sq[mb(mv.from)];
        const int pawn = piece == 1 || piece == 7;
        const int capture = b.sq[mb(mv.to)] != EMPTY || mv.flag == 2;
        play(&b, &mv);
        memcpy(dst, r, (size_t)stride);
        PosRecord *o = (PosRecord *)dst;
        memset(o->pieces, 0, sizeof o->pieces);
        for (int s = 0; s < 64; ++s) {
            int p = b.sq[mb(s)];
            if (p != EMPTY) o->pieces[p - 1] |= 1ULL << s;
        }
        o->stm = (uint8_t)b.stm;
        o->castling = (uint8_t)b.castling;
        o->ep_square = (uint8_t)(b.ep ? sq64(b.ep) : 64);
        o->halfmove = (uint8_t)((pawn || capture) ? 0 : (r->halfmove < 255 ? r->halfmove + 1 : 255));
        o->repetitions = 0;
        if (stride == (int)sizeof(PosRecordH8)) {
            const PosRecordH8 *h = (const PosRecordH8 *)r;
            PosRecordH8 *oh = (PosRecordH8 *)dst;
            for (int t = 6; t >= 1; --t) {
                memcpy(oh->hist_pieces[t], h->hist_pieces[t - 1], sizeof h->hist_pieces[0]);
                oh->hist_rep[t] = h->hist_rep[t - 1];
            }
            memcpy(oh->hist_pieces[0], r->pieces, sizeof r->pieces);
            oh->hist_rep[0] = r->repetitions;
            oh->n_hist = (uint8_t)(h->n_hist < 7 ? h->n_hist + 1 : 7);
        } else if (stride == (int)sizeof(PosRecordM8)) {
            const PosRecordM8 *m = (const PosRecordM8 *)r;
            PosRecordM8 *om = (PosRecordM8 *)dst;
            for (int t = 7; t >= 1; --t) { om->move_from[t] = m->move_from[t - 1]; om->move_to[t] = m->move_to[t - 1]; }
            om->move_from[0] = (uint8_t)mv.from;
            om->move_to[0] = (uint8_t)mv.to;
            om->n_moves = (uint8_t)(m->n_moves < 8 ? m->n_moves + 1 : 8);
        }
    }
    return 0;
}

/* 1 iff the side to move of `record` is in check. */
int orc_in_check(const void *record) {
    MBoard b; load_record((const PosRecord *)record, &b);
    return is_attacked(&b, find_king(&b, b.stm), b.stm ^ 1);
}
