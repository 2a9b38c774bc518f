/*
 * CPU oracle for descriptor-driven batched tensor movement.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, per-element definition of
 * what the CUDA path must produce.  It shares no code, header, table or helper
 * with the CUDA library, and nothing in the product path may call it; only the
 * tests, the smoke check and the CPU-baseline leg of the benchmark do.
 *
 * What the paper fixes (and what it leaves open):
 *   - publish() flushes the KV cache of a request's whole context out of the
 *     engine's paged pool (Table 2, "Instance Operation"; Sec. 3.2; Listing 1),
 *     hydrate() loads it into the destination engine's pool (Table 2; Sec. 4.5
 *     step 8).  Each KV page is one artifact (Sec. 6.3).
 *   - Artifact.view(slice) derives a slice of a tensor, one per tensor-parallel
 *     rank (Table 2; Sec. 6.2); tensor_dict() materialises an artifact into a
 *     compute-ready tensor (Table 2; Sec. 5 "Tensor Materialization and
 *     Transfer"); transform_into() fills a caller-owned target buffer
 *     (Table 2; Sec. 3.2).
 *   - Artifacts are immutable with one canonical content (Sec. 3.2), so every
 *     operation here is an exact byte copy with exactly one correct result.
 *   The paper gives no memory layout; the layouts below are this library's
 *   reading of those operations and are written out as formulas.
 *
 * Layouts (all sizes in elements of E bytes; d is contiguous everywhere):
 *   paged pool, plane (l,c), c=0 for K, c=1 for V, block b, slot n, head h:
 *     NHD: base[l*2+c] + b*block_stride + (((n)*H + h)*D + d)*E + e
 *     HND: base[l*2+c] + b*block_stride + (((h)*B + n)*D + d)*E + e
 *   token t of request r lives in block BT[bt_off[r] + t / B], slot t % B.
 *   packed buffer: requests back to back in request order,
 *     off_0 = 0, off_{r+1} = off_r + L*2*T_r*H*D*E, and inside request r
 *     NHD: off_r + ((((l*2 + c)*T_r + t)*H + h)*D + d)*E + e
 *     HND: off_r + ((((l*2 + c)*H + h)*T_r + t)*D + d)*E + e
 *   Two options of the packed side (a consumer's view of the request, Table 2 "view"):
 *   - head slice [h0, h0+Hs): the packed buffer holds only those heads; H becomes Hs and h
 *     becomes h - h0 in the formulas above (a tensor-parallel consumer owns a head range);
 *   - layer-major order: plane (l,c) of ALL requests is contiguous, so that a consumer can
 *     start on layer 0 while later layers are still in flight:
 *       plane(l,c) = (l*2 + c) * (sum_q T_q) * Hs*D*E,  req_r = (sum_{q<r} T_q) * Hs*D*E
 *       NHD: plane + req_r + ((t*Hs + h')*D + d)*E + e
 *       HND: plane + req_r + ((h'*T_r + t)*D + d)*E + e
 *
 * Every function optionally bumps a per-byte write counter (uint8, saturating)
 * so the tests can prove that each destination byte is written exactly once.
 * Requests [r_begin, r_end) are processed, so that callers may split the work
 * over host threads; the arithmetic is identical for any split.
 */
#include <stddef.h>
#include <stdint.h>

enum { ORACLE_NHD = 0, ORACLE_HND = 1 };

typedef struct {
    int64_t L, B, H, D, E; /* layers, block size (tokens), kv heads, head dim, bytes per element */
} oracle_kv_shape;

typedef struct {
    int32_t layout;       /* ORACLE_NHD or ORACLE_HND, inside one block */
    int64_t block_stride; /* bytes between consecutive blocks of one (l,c) plane */
} oracle_pool_geom;

static void bump(uint8_t *cnt, int64_t a)
{
    if (cnt && cnt[a] != 255) cnt[a]++;
}

/* Byte offset, inside plane (l,c), of byte e of element (b, n, h, d). */
static int64_t pool_off(const oracle_kv_shape *s, const oracle_pool_geom *g,
                        int64_t b, int64_t n, int64_t h, int64_t d, int64_t e)
{
    if (g->layout == ORACLE_NHD)
        return b * g->block_stride + ((n * s->H + h) * s->D + d) * s->E + e;
    return b * g->block_stride + ((h * s->B + n) * s->D + d) * s->E + e;
}

enum { ORACLE_REQUEST_MAJOR = 0, ORACLE_LAYER_MAJOR = 1 };

typedef struct {
    int32_t layout; /* ORACLE_NHD / ORACLE_HND of the packed buffer */
    int32_t order;  /* ORACLE_REQUEST_MAJOR / ORACLE_LAYER_MAJOR */
    int64_t h0, hs; /* head slice [h0, h0 + hs) held by the packed buffer */
} oracle_packed_geom;

/* Byte offset in the packed buffer of byte e of (request r, l, c, token t, head h, d). */
static int64_t packed_addr(const oracle_kv_shape *s, const oracle_packed_geom *pg, int64_t R,
                           const int64_t *T, int64_t r, int64_t l, int64_t c, int64_t t,
                           int64_t h, int64_t d, int64_t e)
{
    int64_t hp = h - pg->h0; /* head index inside the slice */
    int64_t before = 0, total = 0;
    for (int64_t q = 0; q < R; q++) {
        if (q < r) before += T[q];
        total += T[q];
    }
    int64_t inner = (pg->layout == ORACLE_NHD) ? ((t * pg->hs + hp) * s->D + d) * s->E + e
                                               : ((hp * T[r] + t) * s->D + d) * s->E + e;
    int64_t tok = pg->hs * s->D * s->E; /* bytes of one token of one plane */
    if (pg->order == ORACLE_REQUEST_MAJOR)
        return before * s->L * 2 * tok + (l * 2 + c) * T[r] * tok + inner;
    return (l * 2 + c) * total * tok + before * tok + inner;
}

/* publish / offload: gather every valid token of every request into the packed buffer. */
void oracle_kv_pack(const oracle_kv_shape *s, const oracle_pool_geom *g,
                    const uint8_t *const *pool_base, /* [L*2] plane pointers */
                    int64_t R, const int64_t *T, const int64_t *bt_off, const int32_t *bt,
                    const oracle_packed_geom *pg, uint8_t *packed, uint8_t *packed_cnt,
                    int64_t r_begin, int64_t r_end)
{
    for (int64_t r = r_begin; r < r_end; r++)
        for (int64_t l = 0; l < s->L; l++)
            for (int64_t c = 0; c < 2; c++)
                for (int64_t t = 0; t < T[r]; t++) {
                    int64_t b = bt[bt_off[r] + t / s->B], n = t % s->B;
                    for (int64_t h = pg->h0; h < pg->h0 + pg->hs; h++)
                        for (int64_t d = 0; d < s->D; d++)
                            for (int64_t e = 0; e < s->E; e++) {
                                int64_t q = packed_addr(s, pg, R, T, r, l, c, t, h, d, e);
                                packed[q] = pool_base[l * 2 + c][pool_off(s, g, b, n, h, d, e)];
                                bump(packed_cnt, q);
                            }
                }
}

/* hydrate / reload: scatter the packed buffer into the blocks named by the table.
 * pool_cnt, when given, is one counter array per plane. */
void oracle_kv_unpack(const oracle_kv_shape *s, const oracle_pool_geom *g,
                      uint8_t *const *pool_base, uint8_t *const *pool_cnt,
                      int64_t R, const int64_t *T, const int64_t *bt_off, const int32_t *bt,
                      const oracle_packed_geom *pg, const uint8_t *packed,
                      int64_t r_begin, int64_t r_end)
{
    for (int64_t r = r_begin; r < r_end; r++)
        for (int64_t l = 0; l < s->L; l++)
            for (int64_t c = 0; c < 2; c++)
                for (int64_t t = 0; t < T[r]; t++) {
                    int64_t b = bt[bt_off[r] + t / s->B], n = t % s->B;
                    for (int64_t h = pg->h0; h < pg->h0 + pg->hs; h++)
                        for (int64_t d = 0; d < s->D; d++)
                            for (int64_t e = 0; e < s->E; e++) {
                                int64_t p = pool_off(s, g, b, n, h, d, e);
                                pool_base[l * 2 + c][p] = packed[packed_addr(s, pg, R, T, r, l, c, t, h, d, e)];
                                if (pool_cnt) bump(pool_cnt[l * 2 + c], p);
                            }
                }
}

/* publish followed by hydrate, fused: pool to pool through two block tables that
 * share bt_off.  The two pools may differ in layout and block stride (a device
 * pool and a page-first host pool, for instance). */
void oracle_kv_migrate(const oracle_kv_shape *s,
                       const oracle_pool_geom *gs, const uint8_t *const *src_base,
                       const oracle_pool_geom *gd, uint8_t *const *dst_base, uint8_t *const *dst_cnt,
                       int64_t R, const int64_t *T, const int64_t *bt_off,
                       const int32_t *bt_src, const int32_t *bt_dst,
                       int64_t r_begin, int64_t r_end)
{
    (void)R;
    for (int64_t r = r_begin; r < r_end; r++)
        for (int64_t l = 0; l < s->L; l++)
            for (int64_t c = 0; c < 2; c++)
                for (int64_t t = 0; t < T[r]; t++) {
                    int64_t j = bt_off[r] + t / s->B, n = t % s->B;
                    for (int64_t h = 0; h < s->H; h++)
                        for (int64_t d = 0; d < s->D; d++)
                            for (int64_t e = 0; e < s->E; e++) {
                                int64_t p = pool_off(s, gd, bt_dst[j], n, h, d, e);
                                dst_base[l * 2 + c][p] =
                                    src_base[l * 2 + c][pool_off(s, gs, bt_src[j], n, h, d, e)];
                                if (dst_cnt) bump(dst_cnt[l * 2 + c], p);
                            }
                }
}

/*
 * Second, independently written formulation of pack: walk the packed buffer
 * byte by byte, decode which (r,l,c,t,h,d,e) that byte is, and fetch it from
 * the pool.  Used only to cross-check the forward loops above.
 */
void oracle_kv_pack_inverse(const oracle_kv_shape *s, const oracle_pool_geom *g,
                            const uint8_t *const *pool_base,
                            int64_t R, const int64_t *T, const int64_t *bt_off, const int32_t *bt,
                            int32_t packed_layout, uint8_t *packed, int64_t q_begin, int64_t q_end)
{
    int64_t r = 0, start = 0;
    for (int64_t q = q_begin; q < q_end; q++) {
        /* find the request whose region holds byte q */
        while (r < R && q >= start + s->L * 2 * T[r] * s->H * s->D * s->E) {
            start += s->L * 2 * T[r] * s->H * s->D * s->E;
            r++;
        }
        if (r >= R) return;
        int64_t x = q - start;
        int64_t e = x % s->E;  x /= s->E;
        int64_t d = x % s->D;  x /= s->D;
        int64_t t, h;
        if (packed_layout == ORACLE_NHD) { h = x % s->H;  x /= s->H;  t = x % T[r];  x /= T[r]; }
        else                             { t = x % T[r];  x /= T[r];  h = x % s->H;  x /= s->H; }
        int64_t c = x % 2, l = x / 2;
        int64_t b = bt[bt_off[r] + t / s->B], n = t % s->B;
        int64_t within = (g->layout == ORACLE_NHD) ? ((n * s->H + h) * s->D + d)
                                                   : ((h * s->B + n) * s->D + d);
        packed[q] = pool_base[l * 2 + c][b * g->block_stride + within * s->E + e];
    }
}

/*
 * Weight materialisation (tensor_dict / view / transform_into).
 * Tensor i has ndim <= 4 dims shape[i][0..3] (unused dims = 1), E[i] bytes per
 * element, and starts at byte blob_off[i] of the flat blob, row-major, tight.
 * split_dim[i] = -1 copies the whole tensor; otherwise rank `rank` of `world`
 * receives the slab [rank*n/world, (rank+1)*n/world) of that dim.
 * The destination is tensor i's own buffer dst[i], written row-major with the
 * byte strides dst_stride[i][0..3] (so a destination may be a window of a
 * larger target) starting dst_off[i] bytes in.
 *   dst_i[sum_m j_m*dst_stride_m + e] = blob[off_i + lin(k; shape_i)*E + e],
 *   k_m = j_m + (m == split_dim_i ? rank*shape_i[m]/world : 0)
 */
void oracle_weights(int64_t N, const int64_t *blob_off, const int64_t *E,
                    const int64_t (*shape)[4], const int32_t *split_dim,
                    int64_t rank, int64_t world, const uint8_t *blob,
                    uint8_t *const *dst, const int64_t *dst_off, const int64_t (*dst_stride)[4],
                    uint8_t *const *dst_cnt, int64_t i_begin, int64_t i_end)
{
    (void)N;
    for (int64_t i = i_begin; i < i_end; i++) {
        int64_t ext[4], shift[4];
        for (int m = 0; m < 4; m++) {
            ext[m] = shape[i][m];
            shift[m] = 0;
            if (m == split_dim[i]) {
                ext[m] = shape[i][m] / world;
                shift[m] = rank * ext[m];
            }
        }
        for (int64_t j0 = 0; j0 < ext[0]; j0++)
            for (int64_t j1 = 0; j1 < ext[1]; j1++)
                for (int64_t j2 = 0; j2 < ext[2]; j2++)
                    for (int64_t j3 = 0; j3 < ext[3]; j3++) {
                        int64_t k = (((j0 + shift[0]) * shape[i][1] + (j1 + shift[1])) * shape[i][2]
                                     + (j2 + shift[2])) * shape[i][3] + (j3 + shift[3]);
                        int64_t a = dst_off[i] + j0 * dst_stride[i][0] + j1 * dst_stride[i][1]
                                    + j2 * dst_stride[i][2] + j3 * dst_stride[i][3];
                        for (int64_t e = 0; e < E[i]; e++) {
                            dst[i][a + e] = blob[blob_off[i] + k * E[i] + e];
                            if (dst_cnt) bump(dst_cnt[i], a + e);
                        }
                    }
    }
}

/*
 * Integrity checksum folded into weight materialisation (the materialisation pipeline checks
 * integrity, Sec. 5 on tensor materialisation and transfer; the paper does not
 * define the function, this is the library's, stated in its header).
 * Tensor i is read as little-endian 4-byte words x_u at tensor-relative byte offsets 4u:
 *   key(u) = ((u * 0x9E3779B1) << 1 | 1) mod 2^32
 *   sums[i] = sum of x_u * key(u) over the words the rank's slice covers, modulo 2^64.
 * Written byte by byte: the slice is first marked in a byte mask of the tensor, then every
 * fully covered word is added.  A word only partly covered has no defined checksum:
 * *status is set to -1.  mask_scratch must hold the largest tensor's bytes.
 */
void oracle_weights_checksum(int64_t N, const int64_t *blob_off, const int64_t *E,
                             const int64_t (*shape)[4], const int32_t *split_dim,
                             int64_t rank, int64_t world, const uint8_t *blob,
                             uint64_t *sums, uint8_t *mask_scratch, int32_t *status)
{
    *status = 0;
    for (int64_t i = 0; i < N; i++) {
        int64_t ext[4], shift[4], nbytes = E[i];
        for (int m = 0; m < 4; m++) {
            nbytes *= shape[i][m];
            ext[m] = shape[i][m];
            shift[m] = 0;
            if (m == split_dim[i]) {
                ext[m] = shape[i][m] / world;
                shift[m] = rank * ext[m];
            }
        }
        for (int64_t p = 0; p < nbytes; p++) mask_scratch[p] = 0;
        for (int64_t j0 = 0; j0 < ext[0]; j0++)
            for (int64_t j1 = 0; j1 < ext[1]; j1++)
                for (int64_t j2 = 0; j2 < ext[2]; j2++)
                    for (int64_t j3 = 0; j3 < ext[3]; j3++) {
                        int64_t k = (((j0 + shift[0]) * shape[i][1] + (j1 + shift[1])) * shape[i][2]
                                     + (j2 + shift[2])) * shape[i][3] + (j3 + shift[3]);
                        for (int64_t e = 0; e < E[i]; e++) mask_scratch[k * E[i] + e] = 1;
                    }
        uint64_t sum = 0;
        for (int64_t u = 0; u * 4 < nbytes; u++) {
            int covered = 0;
            uint32_t x = 0;
            for (int b = 0; b < 4; b++) {
                int64_t p = u * 4 + b;
                if (p < nbytes && mask_scratch[p]) {
                    covered++;
                    x |= (uint32_t)blob[blob_off[i] + p] << (8 * b);
                }
            }
            if (covered == 4) {
                uint32_t key = (((uint32_t)u * 0x9E3779B1u) << 1) | 1u;
                sum += (uint64_t)x * (uint64_t)key;
            } else if (covered != 0) {
                *status = -1;
            }
        }
        sums[i] = sum;
    }
}
