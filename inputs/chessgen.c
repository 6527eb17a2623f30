/*
 * Seeded synthetic-position generator: random legal playouts from the standard
 * chess start position.
 *
 * This file serves both the CPU oracle and the CUDA library as a source of
 * INPUTS only.  It knows the rules of chess (it must, to play legal plies) but
 * nothing of what the evaluated method computes: no plane encoding, no policy
 * index map, no legal-move mask, no network arithmetic.
 *
 * Board here: a plain 64-entry array, square = file + 8*rank (a1 = 0, h8 = 63).
 * Legality: generate pseudo-legal moves, play each, reject it if the mover's
 * king is then attacked.
 *
 * Recipe (one independent playout per emitted position):
 *   stream  = xoshiro256** seeded by SplitMix64(base_seed XOR index)
 *   n       = lo + next() % (hi - lo + 1)          (ply count of the playout)
 *   each ply: legal moves sorted by (from, to, promotion), pick next() % count
 *   a playout that reaches mate or stalemate before n plies is discarded and
 *   drawn again from the same stream; draw rules never stop a playout.
 * The emitted record holds the final position, its halfmove clock, how many
 * earlier positions of the playout equal it, and the seven boards before it.
 */
#include <stdint.h>
#include <string.h>
#include <stdlib.h>

enum { EMPTY = 0, WP = 1, WN, WB, WR, WQ, WK, BP, BN, BB, BR, BQ, BK };

typedef struct {
    int8_t sq[64];
    uint8_t stm;      /* 0 white to move, 1 black */
    uint8_t castling; /* bit0 white O-O, bit1 white O-O-O, bit2 black O-O, bit3 black O-O-O */
    uint8_t ep;       /* square behind a pawn that just advanced two ranks, else 64 */
    int halfmove;
} Board;

typedef struct {
    uint8_t from, to, promo; /* promo: 0 none, 1 N, 2 B, 3 R, 4 Q */
    uint8_t kind;            /* 0 normal, 1 double push, 2 en passant, 3 castle short, 4 castle long */
} Move;

/* Output record: matches the library's position record with history (784 bytes). */
typedef struct {
    uint64_t pieces[12];
    uint8_t stm, castling, ep_square, halfmove, repetitions, pad[3];
} RecCur;
typedef struct {
    RecCur cur;
    uint64_t hist_pieces[7][12];
    uint8_t hist_rep[7];
    uint8_t n_hist;
} RecH8;

/* Record with the last eight moves instead of the last seven boards (128 bytes): the input of
 * the 52-plane encoder (App. D.1, Table D.1: recent moves as origin / destination squares,
 * castling recorded as the king's own move). */
typedef struct {
    RecCur cur;
    uint8_t move_from[8], move_to[8]; /* absolute squares, most recent move first */
    uint8_t n_moves;                  /* how many of the eight exist */
    uint8_t pad[7];
} RecM8;

/* ---- random stream ------------------------------------------------------- */
typedef struct { uint64_t s[4]; } Rng;
static uint64_t splitmix64(uint64_t *x) {
    uint64_t z = (*x += 0x9E3779B97F4A7C15ULL);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}
static void rng_seed(Rng *r, uint64_t seed) {
    for (int i = 0; i < 4; ++i) r->s[i] = splitmix64(&seed);
}
static inline uint64_t rotl(uint64_t x, int k) { return (x << k) | (x >> (64 - k)); }
static uint64_t rng_next(Rng *r) {
    uint64_t *s = r->s;
    uint64_t result = rotl(s[1] * 5, 7) * 9;
    uint64_t t = s[1] << 17;
    s[2] ^= s[0]; s[3] ^= s[1]; s[1] ^= s[2]; s[0] ^= s[3];
    s[2] ^= t; s[3] = rotl(s[3], 45);
    return result;
}

/* ---- rules ---------------------------------------------------------------- */
static inline int is_white(int p) { return p >= WP && p <= WK; }
static inline int is_black(int p) { return p >= BP; }
static inline int side_of(int p) { return p == EMPTY ? -1 : (p >= BP); }

static void board_start(Board *b) {
    static const int8_t back[8] = { WR, WN, WB, WQ, WK, WB, WN, WR };
    memset(b->sq, 0, sizeof b->sq);
    for (int f = 0; f < 8; ++f) {
        b->sq[f] = back[f];
        b->sq[8 + f] = WP;
        b->sq[48 + f] = BP;
        b->sq[56 + f] = (int8_t)(back[f] + 6);
    }
    b->stm = 0; b->castling = 15; b->ep = 64; b->halfmove = 0;
}

static const int KN[8][2] = { {1,2},{2,1},{2,-1},{1,-2},{-1,-2},{-2,-1},{-2,1},{-1,2} };
static const int KG[8][2] = { {0,1},{1,1},{1,0},{1,-1},{0,-1},{-1,-1},{-1,0},{-1,1} };

/* Is square s attacked by a piece of colour `by` (0 white, 1 black)? */
static int attacked(const Board *b, int s, int by) {
    int f = s & 7, r = s >> 3;
    int pawn = by ? BP : WP, knight = by ? BN : WN, bishop = by ? BB : WB;
    int rook = by ? BR : WR, queen = by ? BQ : WQ, king = by ? BK : WK;
    /* pawns: a white pawn on (f±1, r-1) attacks (f, r) */
    int pr = by ? r + 1 : r - 1;
    if (pr >= 0 && pr < 8) {
        if (f > 0 && b->sq[pr * 8 + f - 1] == pawn) return 1;
        if (f < 7 && b->sq[pr * 8 + f + 1] == pawn) return 1;
    }
    for (int i = 0; i < 8; ++i) {
        int nf = f + KN[i][0], nr = r + KN[i][1];
        if (nf >= 0 && nf < 8 && nr >= 0 && nr < 8 && b->sq[nr * 8 + nf] == knight) return 1;
        nf = f + KG[i][0]; nr = r + KG[i][1];
        if (nf >= 0 && nf < 8 && nr >= 0 && nr < 8 && b->sq[nr * 8 + nf] == king) return 1;
    }
    for (int i = 0; i < 8; ++i) {
        int df = KG[i][0], dr = KG[i][1];
        int diag = (df != 0 && dr != 0);
        int nf = f + df, nr = r + dr;
        while (nf >= 0 && nf < 8 && nr >= 0 && nr < 8) {
            int p = b->sq[nr * 8 + nf];
            if (p != EMPTY) {
                if (p == queen || p == (diag ? bishop : rook)) return 1;
                break;
            }
            nf += df; nr += dr;
        }
    }
    return 0;
}

static int king_square(const Board *b, int side) {
    int k = side ? BK : WK;
    for (int s = 0; s < 64; ++s) if (b->sq[s] == k) return s;
    return -1;
}

static void make_move(Board *b, Move m) {
    int p = b->sq[m.from];
    int cap = b->sq[m.to];
    int us = b->stm;
    int pawn_move = (p == WP || p == BP);
    b->sq[m.from] = EMPTY;
    b->sq[m.to] = (int8_t)p;
    if (m.kind == 2) {               /* en passant: captured pawn is beside the origin */
        int cs = (m.to & 7) + 8 * (m.from >> 3);
        b->sq[cs] = EMPTY; cap = 1;
    } else if (m.kind == 3) {        /* short castle */
        int r0 = us ? 56 : 0;
        b->sq[r0 + 7] = EMPTY; b->sq[r0 + 5] = (int8_t)(us ? BR : WR);
    } else if (m.kind == 4) {        /* long castle */
        int r0 = us ? 56 : 0;
        b->sq[r0 + 0] = EMPTY; b->sq[r0 + 3] = (int8_t)(us ? BR : WR);
    }
    if (m.promo) {
        static const int8_t wp[5] = { 0, WN, WB, WR, WQ };
        b->sq[m.to] = (int8_t)(wp[m.promo] + (us ? 6 : 0));
    }
    /* castling rights: lost when king or rook leaves, or a rook is captured at home */
    if (p == WK) b->castling &= (uint8_t)~3;
    if (p == BK) b->castling &= (uint8_t)~12;
    if (m.from == 7 || m.to == 7) b->castling &= (uint8_t)~1;
    if (m.from == 0 || m.to == 0) b->castling &= (uint8_t)~2;
    if (m.from == 63 || m.to == 63) b->castling &= (uint8_t)~4;
    if (m.from == 56 || m.to == 56) b->castling &= (uint8_t)~8;
    b->ep = (m.kind == 1) ? (uint8_t)((m.from + m.to) / 2) : 64;
    b->halfmove = (pawn_move || cap != EMPTY) ? 0 : b->halfmove + 1;
    b->stm ^= 1;
}

static int add_move(Move *list, int n, int from, int to, int promo, int kind) {
    list[n].from = (uint8_t)from; list[n].to = (uint8_t)to;
    list[n].promo = (uint8_t)promo; list[n].kind = (uint8_t)kind;
    return n + 1;
}

static int pseudo_moves(const Board *b, Move *list) {
    int n = 0, us = b->stm;
    for (int s = 0; s < 64; ++s) {
        int p = b->sq[s];
        if (p == EMPTY || side_of(p) != us) continue;
        int f = s & 7, r = s >> 3;
        int t = us ? p - 6 : p; /* 1..6 */
        if (t == WP) {
            int dir = us ? -1 : 1, start = us ? 6 : 1, last = us ? 0 : 7;
            int nr = r + dir;
            if (nr < 0 || nr > 7) continue;
            int fwd = nr * 8 + f;
            if (b->sq[fwd] == EMPTY) {
                if (nr == last) for (int q = 1; q <= 4; ++q) n = add_move(list, n, s, fwd, q, 0);
                else {
                    n = add_move(list, n, s, fwd, 0, 0);
                    if (r == start && b->sq[fwd + dir * 8] == EMPTY)
                        n = add_move(list, n, s, fwd + dir * 8, 0, 1);
                }
            }
            for (int df = -1; df <= 1; df += 2) {
                int nf = f + df;
                if (nf < 0 || nf > 7) continue;
                int to = nr * 8 + nf, q = b->sq[to];
                if (q != EMPTY && side_of(q) != us) {
                    if (nr == last) for (int k = 1; k <= 4; ++k) n = add_move(list, n, s, to, k, 0);
                    else n = add_move(list, n, s, to, 0, 0);
                } else if (q == EMPTY && to == b->ep && b->ep < 64) {
                    n = add_move(list, n, s, to, 0, 2);
                }
            }
        } else if (t == WN || t == WK) {
            const int (*d)[2] = (t == WN) ? KN : KG;
            for (int i = 0; i < 8; ++i) {
                int nf = f + d[i][0], nr = r + d[i][1];
                if (nf < 0 || nf > 7 || nr < 0 || nr > 7) continue;
                int q = b->sq[nr * 8 + nf];
                if (q == EMPTY || side_of(q) != us) n = add_move(list, n, s, nr * 8 + nf, 0, 0);
            }
            if (t == WK) {
                int r0 = us ? 56 : 0, them = us ^ 1;
                int ks = us ? 4 : 1, qs = us ? 8 : 2;
                int rook = us ? BR : WR;
                if (s == r0 + 4 && !attacked(b, s, them)) {
                    if ((b->castling & ks) && b->sq[r0 + 7] == rook &&
                        b->sq[r0 + 5] == EMPTY && b->sq[r0 + 6] == EMPTY &&
                        !attacked(b, r0 + 5, them) && !attacked(b, r0 + 6, them))
                        n = add_move(list, n, s, r0 + 6, 0, 3);
                    if ((b->castling & qs) && b->sq[r0] == rook &&
                        b->sq[r0 + 1] == EMPTY && b->sq[r0 + 2] == EMPTY && b->sq[r0 + 3] == EMPTY &&
                        !attacked(b, r0 + 3, them) && !attacked(b, r0 + 2, them))
                        n = add_move(list, n, s, r0 + 2, 0, 4);
                }
            }
        } else {
            for (int i = 0; i < 8; ++i) {
                int df = KG[i][0], dr = KG[i][1];
                int diag = (df != 0 && dr != 0);
                if (t == WB && !diag) continue;
                if (t == WR && diag) continue;
                int nf = f + df, nr = r + dr;
                while (nf >= 0 && nf < 8 && nr >= 0 && nr < 8) {
                    int q = b->sq[nr * 8 + nf];
                    if (q == EMPTY) n = add_move(list, n, s, nr * 8 + nf, 0, 0);
                    else { if (side_of(q) != us) n = add_move(list, n, s, nr * 8 + nf, 0, 0); break; }
                    nf += df; nr += dr;
                }
            }
        }
    }
    return n;
}

static int legal_moves(const Board *b, Move *out) {
    Move tmp[256];
    int n = pseudo_moves(b, tmp), k = 0;
    for (int i = 0; i < n; ++i) {
        Board c = *b;
        make_move(&c, tmp[i]);
        if (!attacked(&c, king_square(&c, b->stm), b->stm ^ 1)) out[k++] = tmp[i];
    }
    return k;
}

static int move_key(const Move *m) { return (m->from << 16) | (m->to << 8) | m->promo; }
static int cmp_move(const void *a, const void *b) {
    return move_key((const Move *)a) - move_key((const Move *)b);
}

/* ---- record writing -------------------------------------------------------- */
static void board_bitboards(const Board *b, uint64_t bb[12]) {
    for (int i = 0; i < 12; ++i) bb[i] = 0;
    for (int s = 0; s < 64; ++s) if (b->sq[s]) bb[b->sq[s] - 1] |= 1ULL << s;
}
static int same_position(const Board *a, const Board *b) {
    return a->stm == b->stm && a->castling == b->castling && a->ep == b->ep &&
           memcmp(a->sq, b->sq, 64) == 0;
}

#define MAX_PLIES 1024

/*
 * Writes `count` records (784 bytes each) for position indices
 * first_index .. first_index+count-1.  Even indices draw their ply count from
 * [lo_even, hi_even], odd ones from [lo_odd, hi_odd].  plies_out (optional)
 * receives each record's ply count.  Returns 0, or -1 on bad arguments.
 */
static int play_one(uint64_t base_seed, int64_t index, int lo_even, int hi_even, int lo_odd, int hi_odd,
                    Board *game, int *reps, Move *played)
{
    Rng rng; rng_seed(&rng, base_seed ^ (uint64_t)index);
    int lo = (index & 1) ? lo_odd : lo_even, hi = (index & 1) ? hi_odd : hi_even;
    int n;
    for (;;) {
        n = lo + (int)(rng_next(&rng) % (uint64_t)(hi - lo + 1));
        board_start(&game[0]); reps[0] = 0;
        int ply = 0, ok = 1;
        Move list[256];
        for (; ply < n; ++ply) {
            int k = legal_moves(&game[ply], list);
            if (k == 0) { ok = 0; break; }
            qsort(list, (size_t)k, sizeof(Move), cmp_move);
            Move m = list[rng_next(&rng) % (uint64_t)k];
            played[ply] = m;
            game[ply + 1] = game[ply];
            make_move(&game[ply + 1], m);
            int r = 0;
            for (int j = 0; j <= ply; ++j) r += same_position(&game[j], &game[ply + 1]);
            reps[ply + 1] = r;
        }
        if (ok) {
            Move tmp[256];
            if (legal_moves(&game[n], tmp) > 0) break; /* emitted positions are never terminal */
        }
    }
    return n;
}

static void fill_cur(RecCur *cur, const Board *b, int reps)
{
    board_bitboards(b, cur->pieces);
    cur->stm = b->stm;
    cur->castling = b->castling;
    cur->ep_square = b->ep;
    cur->halfmove = (uint8_t)(b->halfmove > 255 ? 255 : b->halfmove);
    cur->repetitions = (uint8_t)(reps > 255 ? 255 : reps);
}

static int generate(uint64_t base_seed, int64_t first_index, int count,
                    int lo_even, int hi_even, int lo_odd, int hi_odd,
                    void *records_out, int32_t *plies_out, int with_moves)
{
    if (count < 0 || !records_out || lo_even < 0 || lo_odd < 0 || hi_even < lo_even ||
        hi_odd < lo_odd || hi_even >= MAX_PLIES || hi_odd >= MAX_PLIES) return -1;
    Board *game = (Board *)malloc(sizeof(Board) * (MAX_PLIES + 1));
    int *reps = (int *)malloc(sizeof(int) * (MAX_PLIES + 1));
    Move *played = (Move *)malloc(sizeof(Move) * (MAX_PLIES + 1));
    if (!game || !reps || !played) { free(game); free(reps); free(played); return -1; }
    for (int i = 0; i < count; ++i) {
        int n = play_one(base_seed, first_index + i, lo_even, hi_even, lo_odd, hi_odd, game, reps, played);
        if (with_moves) {
            RecM8 *rec = &((RecM8 *)records_out)[i];
            memset(rec, 0, sizeof *rec);
            fill_cur(&rec->cur, &game[n], reps[n]);
            int nm = n < 8 ? n : 8;
            rec->n_moves = (uint8_t)nm;
            for (int t = 0; t < nm; ++t) {
                rec->move_from[t] = played[n - 1 - t].from;
                rec->move_to[t] = played[n - 1 - t].to;
            }
        } else {
            RecH8 *rec = &((RecH8 *)records_out)[i];
            memset(rec, 0, sizeof *rec);
            fill_cur(&rec->cur, &game[n], reps[n]);
            int nh = n < 7 ? n : 7;
            rec->n_hist = (uint8_t)nh;
            for (int t = 1; t <= nh; ++t) {
                board_bitboards(&game[n - t], rec->hist_pieces[t - 1]);
                rec->hist_rep[t - 1] = (uint8_t)(reps[n - t] > 255 ? 255 : reps[n - t]);
            }
        }
        if (plies_out) plies_out[i] = n;
    }
    free(game); free(reps); free(played);
    return 0;
}

int azgen_positions(uint64_t base_seed, int64_t first_index, int count,
                    int lo_even, int hi_even, int lo_odd, int hi_odd,
                    void *records_out, int32_t *plies_out)
{
    return generate(base_seed, first_index, count, lo_even, hi_even, lo_odd, hi_odd, records_out, plies_out, 0);
}

/* The same positions (same seeds, same playouts) as 128-byte records with the last eight moves. */
int azgen_positions_moves(uint64_t base_seed, int64_t first_index, int count,
                          int lo_even, int hi_even, int lo_odd, int hi_odd,
                          void *records_out, int32_t *plies_out)
{
    return generate(base_seed, first_index, count, lo_even, hi_even, lo_odd, hi_odd, records_out, plies_out, 1);
}

/* Legal moves of one 104-byte position record, sorted by (from, to, promotion);
 * moves_out holds up to 256 triples (from, to, promo); castling is reported as
 * the king's own move (e1g1 / e1c1).  Used by tests to cross-check generators. */
int azgen_legal_moves(const void *record, uint8_t *moves_out)
{
    const RecCur *rc = (const RecCur *)record;
    Board b; memset(b.sq, 0, 64);
    for (int p = 0; p < 12; ++p)
        for (int s = 0; s < 64; ++s) if ((rc->pieces[p] >> s) & 1) b.sq[s] = (int8_t)(p + 1);
    b.stm = rc->stm; b.castling = rc->castling; b.ep = rc->ep_square; b.halfmove = rc->halfmove;
    Move list[256];
    int k = legal_moves(&b, list);
    qsort(list, (size_t)k, sizeof(Move), cmp_move);
    for (int i = 0; i < k; ++i) {
        moves_out[3 * i] = list[i].from; moves_out[3 * i + 1] = list[i].to; moves_out[3 * i + 2] = list[i].promo;
    }
    return k;
}

int azgen_record_bytes(void) { return (int)sizeof(RecH8); }
int azgen_move_record_bytes(void) { return (int)sizeof(RecM8); }
