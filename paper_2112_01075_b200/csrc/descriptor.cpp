// From two layouts of the same global array to the copy descriptor a kernel receives, and from a
// synthesized sequence to the list of kernel launches (one per collective, or one per fused run
// of adjacent collectives -- merging of adjacent operations, Section 7.1, taken one step further:
// on one GPU any run of steps composes into a single strided copy).
#include <algorithm>
#include <numeric>

#include "plan.hpp"

namespace redist {

namespace {

FastDiv make_div(uint32_t d)
{
    FastDiv f{d, 0, 0};
    if (d > 1) {
        uint32_t lg = 0;
        while ((1ull << lg) < d) ++lg;                 // ceil(log2 d)
        const uint32_t pw = 31 + lg;
        f.mul = uint32_t(((1ull << pw) + d - 1) / d);  // ceil(2^pw / d) < 2^32 because d > 2^(lg-1)
        f.shr = pw - 32;
    }
    return f;
}

i64 round_up(i64 v, i64 a) { return (v + a - 1) / a * a; }

struct RowDigit {
    i64 n, b1, b2;
};

}  // namespace

redist_status build_copy(const Plan &p, const Layout &a, const Layout &b, Launch &out)
{
    const int r = p.rank;
    const i64 e = p.elem_bytes;
    std::vector<i64> g(r), m1(r), m2(r), nq(r), es1(r), es2(r), ts1(r), ts2(r);
    for (int k = r - 1; k >= 0; --k) {
        g[k] = std::gcd(a.tile[k], b.tile[k]);
        m1[k] = a.tile[k] / g[k];
        m2[k] = b.tile[k] / g[k];
        nq[k] = p.global_shape[k] / g[k];
        es1[k] = k == r - 1 ? 1 : es1[k + 1] * a.tile[k + 1];
        es2[k] = k == r - 1 ? 1 : es2[k + 1] * b.tile[k + 1];
        ts1[k] = k == r - 1 ? 1 : ts1[k + 1] * a.ntiles[k + 1];
        ts2[k] = k == r - 1 ? 1 : ts2[k + 1] * b.ntiles[k + 1];
    }
    int kp = -1;   // last dimension whose tile size differs between the two layouts
    for (int k = 0; k < r; ++k)
        if (a.tile[k] != b.tile[k]) kp = k;
    i64 run_elems = 1;
    for (int k = std::max(kp, 0); k < r; ++k) run_elems *= (k == kp ? g[k] : a.tile[k]);
    if (kp < 0) {
        run_elems = 1;
        for (int k = 0; k < r; ++k) run_elems *= a.tile[k];
    }
    i64 run_bytes = run_elems * e;

    CopyGeometry &G = out.geo;
    G = CopyGeometry();
    // unit digits, outer to inner
    i64 n_boxes = 1;
    uint32_t nu = 0;
    for (int k = 0; k < r; ++k) {
        if (nq[k] == 1) continue;
        if (nq[k] >= (1ll << 31) || ts1[k] >= (1ll << 31) || ts2[k] >= (1ll << 31)) return REDIST_EUNSUPPORTED;
        G.unit_n[nu] = make_div(uint32_t(nq[k]));
        G.unit_m1[nu] = make_div(uint32_t(m1[k]));
        G.unit_m2[nu] = make_div(uint32_t(m2[k]));
        G.unit_ts1[nu] = uint32_t(ts1[k]);
        G.unit_ts2[nu] = uint32_t(ts2[k]);
        G.unit_b1[nu] = g[k] * es1[k] * e;
        G.unit_b2[nu] = g[k] * es2[k] * e;
        G.unit_mul[nu] = 1;
        n_boxes *= nq[k];
        if (n_boxes >= (1ll << 31)) return REDIST_EUNSUPPORTED;
        ++nu;
    }
    G.n_unit = nu;
    // short runs: the units of dimension kp that lie in the same source or target tile row become
    // the fastest-varying part of the item number (see copy_params.h)
    G.inner_n = make_div(1);
    G.inner_digit = 0xffffffffu;
    G.inner_span = 1;
    G.inner_mul = 1;
    i64 inner = 1;
    const i64 kInnerRun = 16384;   // runs below this many bytes get adjacent-piece item numbering (measured)
    if (kp >= 0 && run_bytes < kInnerRun && nq[kp] > 1 && m1[kp] * m2[kp] > 1) {
        inner = m1[kp] * m2[kp];
        uint32_t u = 0;
        for (int k = 0; k < kp; ++k)
            if (nq[k] != 1) ++u;
        G.inner_digit = u;
        G.inner_span = uint32_t(inner);
        G.inner_n = make_div(uint32_t(inner));
        G.unit_n[u] = make_div(uint32_t(nq[kp] / inner));
        n_boxes /= inner;
    }
    // Unit digits whose units sit side by side within a few cache lines of a tile (m > 1 and a byte stride
    // below kFastStride on that side) are moved to the end of the digit list: they become the fastest
    // part of the box number, and -- see decode_box -- vary faster than the row groups of a box, so that the
    // blocks which share those lines run at the same time and partial sectors merge in L2.
    const i64 kFastStride = 16384;
    G.fast_boxes = make_div(1);
    {
        std::vector<uint32_t> slow, fast;
        for (uint32_t u = 0; u < nu; ++u) {
            const bool f = u != G.inner_digit && G.unit_n[u].d > 1 &&
                           ((G.unit_m2[u].d > 1 && G.unit_b2[u] < kFastStride) || (G.unit_m1[u].d > 1 && G.unit_b1[u] < kFastStride));
            (f ? fast : slow).push_back(u);
        }
        if (!fast.empty()) {
            CopyGeometry T = G;
            uint32_t pos = 0;
            i64 nfast = 1;
            auto put = [&](uint32_t u) {
                G.unit_n[pos] = T.unit_n[u];
                G.unit_m1[pos] = T.unit_m1[u];
                G.unit_m2[pos] = T.unit_m2[u];
                G.unit_ts1[pos] = T.unit_ts1[u];
                G.unit_ts2[pos] = T.unit_ts2[u];
                G.unit_b1[pos] = T.unit_b1[u];
                G.unit_b2[pos] = T.unit_b2[u];
                G.unit_mul[pos] = T.unit_mul[u];
                if (u == T.inner_digit) G.inner_digit = pos;
                ++pos;
            };
            for (uint32_t u : slow) put(u);
            for (uint32_t u : fast) {
                nfast *= T.unit_n[u].d;
                put(u);
            }
            G.fast_boxes = make_div(uint32_t(nfast));
        }
    }
    // row digits inside a box: the dimensions before kp, merged where both sides stay contiguous
    std::vector<RowDigit> rows;
    for (int k = 0; k < kp; ++k) {
        if (g[k] == 1) continue;
        RowDigit d{g[k], es1[k] * e, es2[k] * e};
        rows.push_back(d);
    }
    for (size_t q = rows.size(); q-- > 1;) {
        RowDigit &o = rows[q - 1], &in = rows[q];
        if (o.b1 == in.n * in.b1 && o.b2 == in.n * in.b2) {
            in.n *= o.n;
            rows.erase(rows.begin() + (q - 1));
        }
    }
    // vector width: the largest power of two dividing every byte quantity that forms an address
    i64 align = 16;
    auto fit = [&](i64 v) {
        while (align > 1 && v % align) align >>= 1;
    };
    fit(run_bytes);
    for (uint32_t u = 0; u < nu; ++u) {
        if (G.unit_m1[u].d > 1) fit(G.unit_b1[u]);
        if (G.unit_m2[u].d > 1) fit(G.unit_b2[u]);
    }
    for (const RowDigit &d : rows) {
        fit(d.b1);
        fit(d.b2);
    }
    const i64 vec = align;
    if (rows.size() > size_t(kMaxRowDigits)) return REDIST_EUNSUPPORTED;
    i64 n_rows = 1;
    for (size_t q = 0; q < rows.size(); ++q) {
        if (rows[q].n >= (1ll << 31)) return REDIST_EUNSUPPORTED;
        G.row_n[q] = make_div(uint32_t(rows[q].n));
        G.row_b1[q] = rows[q].b1;
        G.row_b2[q] = rows[q].b2;
        n_rows *= rows[q].n;
        if (n_rows >= (1ll << 31)) return REDIST_EUNSUPPORTED;
    }
    G.n_row = uint32_t(rows.size());
    G.n_row_tab = G.n_row;
    G.tab_inner = make_div(1);
    G.units_per_run = make_div(1);
    G.unit_bytes = uint32_t(vec);
    G.aligned = vec == 16 ? 1u : 0u;
    G.run_bytes = uint64_t(run_bytes);
    G.rows = uint32_t(n_rows);
    // work items: about 32 KiB read each -- less when every byte read is stored to several
    // replicas, so that the bytes written per block stay comparable
    const Tuning &tune = p.tuning;
    const i64 kItemKb = tune.item_kb > 0 ? tune.item_kb : 0;
    i64 fan = 1;
    if (!b.shared_global) {
        i64 nt = 1;
        for (int k = 0; k < r; ++k) nt *= b.ntiles[k];
        fan = p.n_devices / nt;
    }
    // (the 256-thread kernels: 32 KiB up to fan-out 3, 16 KiB up to 7, 8 KiB from 8.  Every thread of a block
    // decodes the item, so small items pay for it dearly: measured on eleven fan-out problems of the odd-shape
    // sweep, 16 -> 32 KiB at fan-out 2: 4.34-5.07 -> 5.12-6.51 TB/s; 8 -> 16 KiB at fan-out 4: 4.69-5.57 ->
    // 6.07-6.28; at fan-out 8, 8 KiB stays best: 5.74 against 5.17)
    const i64 kItemBytes = kItemKb > 0 ? kItemKb * 1024 : (fan >= 8 ? 8 : fan >= 4 ? 16 : 32) * 1024;
    // Items of the plain bulk-copy kernels: measured best at 20 KiB (12 / 6 KiB for fan-out >= 2 / >= 4) once
    // the kernels wait for their predecessor only after decoding the item -- finer tail, more blocks ready
    // behind the wait.
    const i64 kBulkItemKb = 20;
    // aligned segments of 512 bytes or more go through the bulk-copy kernels (at most one segment per
    // thread, the item staged in at most 47 KiB of shared memory)
    const bool kBulk = tune.bulk > 0;     // 0 keeps every run on the register kernels
    const i64 kBulkMin = 512;             // shortest segment moved by a bulk copy
    const i64 max_chunks = run_bytes / 16;           // whole 16-byte chunks a run can hold
    if (max_chunks >= (1ll << 31)) return REDIST_EUNSUPPORTED;
    const i64 bulk_item_bytes = kItemKb == 0 && kBulk && G.aligned && run_bytes >= kBulkMin
                                    ? (fan >= 4 ? kBulkItemKb * 3 / 10 : fan >= 2 ? kBulkItemKb * 6 / 10 : kBulkItemKb) * 1024
                                    : kItemBytes;
    i64 ipb;
    G.lanes = kBlockThreads;
    G.rows_per_pass = 1;
    bool ragged_bulk = false;
    // gather walk: short runs whose m pieces interleave on one side; the target bytes of a table row
    // (the stretch) are produced in whole 16-byte chunks
    // 0 disables the gather walk, 2 uses it wherever it applies; the default (1) keeps it to the cases
    // where it was measured faster than the walk over unit pieces
    const int kGather = int(tune.gather);
    int g_levels = -1;
    i64 g_stretch = 0;
    if (kGather > 0 && run_bytes < 256 && G.inner_digit != 0xffffffffu && (m1[kp] == 1 || m2[kp] == 1)) {
        const bool long_dst = m2[kp] > 1;
        const i64 m = std::max(m1[kp], m2[kp]);
        const i64 piece_stride = long_dst ? G.unit_b2[G.inner_digit] : G.unit_b1[G.inner_digit];
        i64 S = long_dst ? m * run_bytes : run_bytes;
        int lv = 0;
        for (size_t q = rows.size(); q-- > 0 && lv < kMaxGatherLevels;) {
            if (rows[q].b2 != S || S * rows[q].n >= (1ll << 31)) break;
            S *= rows[q].n;
            ++lv;
        }
        // measured: pays when the target has the long rows and either every chunk is stored to several
        // replicas or the runs are short and come from few tiles; long source rows read badly this way
        const bool pays = long_dst && (fan >= 2 || (run_bytes < 100 && m <= 4));
        if (piece_stride == run_bytes && S >= 32 && (long_dst || lv > 0) && (kGather >= 2 || pays)) {
            g_levels = lv;
            g_stretch = S;
        }
    }
    // zip: the same interleaving when the innermost row digit is contiguous on both sides -- the source
    // segments of an item are then long enough for bulk copies into shared memory
    // 0 disables the zip kernels, 1 uses them only where the gather walk is not chosen; the default (2)
    // wherever they apply (measured: within 0.3 % of the best choice per problem on the odd-shape sweep)
    const int kZip = int(tune.zip);
    const i64 kZipMinRange = 128;         // shortest target range of a table row
    // runs below this many bytes may take the zip and super-box kernels: measured, from 2 KiB the plain bulk
    // copy (aligned runs) and the ragged chunk walk are faster; with units of 1 or 2 bytes (8 or 16 of them to a
    // chunk) the ragged chunk walk, which shifts whole chunks whatever the unit, wins from 512 bytes unless
    // every chunk is stored to four or more replicas
    const i64 kZipRun = vec >= 4 || fan >= 4 ? 2048 : 512;
    const bool zip_run_ok = run_bytes < kZipRun;
    i64 zip_n = 0;
    if (kZip > 0 && kBulk && (kZip >= 2 || g_levels < 0) && zip_run_ok && G.inner_digit != 0xffffffffu &&
        (m1[kp] == 1 || m2[kp] == 1) && !rows.empty()) {
        const bool long_dst = m2[kp] > 1;
        const i64 m = std::max(m1[kp], m2[kp]);
        const i64 piece_stride = long_dst ? G.unit_b2[G.inner_digit] : G.unit_b1[G.inner_digit];
        const RowDigit &d = rows.back();
        const i64 bs = long_dst ? run_bytes : m * run_bytes, bd = long_dst ? m * run_bytes : run_bytes;
        // a source segment of a full item should be worth a bulk copy
        // (one row of the zipped digit must fit the item's shared-memory tile: m segments of a run each, or one
        // segment of a long row; with up to 16 tiles and runs below 2 KiB it always does.  17 to 64 tiles, measured
        // on 32: target rows zipped from 32 tiles and stored to 32 replicas 2.2-3.7 -> 5.3-5.5 TB/s against the
        // ragged chunk walk; long source rows unzipped into 32 tiles 3.8-4.5 -> 5.6-5.7 on runs of 260-372 bytes,
        // but 0.94x from 512 bytes, where the ragged chunk walk stays)
        const i64 one_row = (long_dst ? m : 1) * ((long_dst ? run_bytes : m * run_bytes) + 48);
        if (piece_stride == run_bytes && d.b1 == bs && d.b2 == bd && d.n * bs >= 256 && d.n * bd >= kZipMinRange && m <= 64 &&
            one_row <= 38 * 1024 && (m <= 16 || long_dst || run_bytes < 512))
            zip_n = d.n;
    }
    // box: the item is a super-box -- lcm(source tile, target tile) indices in each of the innermost
    // differing dimensions ("inner" dimensions, kp and as many before it as it takes to make the
    // contiguous pieces on both sides long), times a block of rows of the dimension K just outside them.
    // Source bytes: one contiguous segment per source tile touched; target bytes: one contiguous range
    // per target tile touched.  Chosen (tuning value "box": 0 never, 2 wherever it applies) for short
    // runs where the zip kernels do not apply or would produce target ranges of a few hundred bytes.
    struct BoxDim {
        int k;
        i64 c1, c2, E;
    };
    std::vector<BoxDim> bxd;      // inner dimensions, outer to inner
    int bxK = -2;                 // the dimension outside them (-1: none)
    i64 bx_s1 = 0, bx_s2 = 0, bx_cnt = 0, bx_gK = 1, bx_rpi = 1;
    const i64 kBoxTile = 38 * 1024;
    if (tune.box > 0 && kBulk && kp >= 0 && zip_run_ok && nq[kp] > 1) {
        i64 trail = e;                               // bytes of the identical trailing dimensions
        for (int k = kp + 1; k < r; ++k) trail *= a.tile[k];
        i64 s1 = trail, s2 = trail, sup = trail, n1 = 1, n2 = 1;
        bool ok = true;
        int k = kp;
        while (ok) {
            const i64 c1 = a.tile[k], c2 = b.tile[k];
            if (c1 % c2 != 0 && c2 % c1 != 0) ok = false;      // neither tile size divides the other: not separable
            const i64 E = std::max(c1, c2);
            // (the table of unit places covers one target row; beyond the innermost dimension it has to stay a
            // quarter of an item at most, or tabulating it costs more than walking the item: measured 5.6 ->
            // 3.7 TB/s with a table as long as the item)
            if (ok && (sup * E > kBoxTile || n1 * (E / c1) > kBoxSegments / 4 || n2 * (E / c2) > kBoxSegments / 4 ||
                       s2 * c2 / vec > 4096 || (!bxd.empty() && s2 * c2 > kItemBytes / 4)))
                ok = false;
            if (!ok) break;
            bxd.insert(bxd.begin(), BoxDim{k, c1, c2, E});
            s1 *= c1;
            s2 *= c2;
            sup *= E;
            n1 *= E / c1;
            n2 *= E / c2;
            // long enough with the rows of the next dimension out?  (Segments and ranges of 2 KiB: every range
            // costs a lane group some forty instructions of set-up and a ragged head and tail, measured 3.7 ->
            // 5+ TB/s on ranges of 616 bytes made 16 KiB.  An item is filled up with further outer rows, so
            // the inner dimensions need not grow for the sake of its size.)
            const i64 gk = k > 0 ? g[k - 1] : 1;
            const i64 cmax = std::min<i64>(gk, std::max<i64>(1, kItemBytes / sup));
            if (std::min(s1, s2) * cmax >= 2048 || k == 0 || int(bxd.size()) == kMaxBoxDims) break;
            --k;
        }
        if (!bxd.empty() && (ok || int(bxd.size()) > 0)) {
            // (a failed extension keeps what was accepted so far)
            bxK = bxd.front().k - 1;
            bx_gK = bxK >= 0 ? g[bxK] : 1;
            bx_s1 = s1;
            bx_s2 = s2;
            i64 cnt = std::max<i64>(1, std::min<i64>(bx_gK, kItemBytes / sup));
            while (cnt > 1 && n1 * (round_up(cnt * s1, 16) + 32) > kBoxTile) --cnt;
            bx_cnt = cnt;
            // outer rows per item: fill the item up, within the segment and range tables and the tile
            i64 outer_rows = 1;
            for (int q = 0; q < bxK; ++q) outer_rows *= g[q];
            const i64 seg_pitch = round_up(cnt * s1, 16) + 32;
            i64 rpi = std::max<i64>(1, kItemBytes / (cnt * sup));
            rpi = std::min<i64>(std::min<i64>(rpi, outer_rows), std::min<i64>(kBoxRows, kBoxSegments / std::max(n1, n2)));
            rpi = std::max<i64>(1, std::min<i64>(rpi, kBoxTile / (seg_pitch * n1)));
            bx_rpi = rpi;
            // (staged segments within the tile; with the table of places and the static tables of the kernel
            // the block stays below the 48 KiB a launch gets without opting in to more)
            const bool fits = rpi * n1 * seg_pitch <= kBoxTile && rpi * n1 * seg_pitch + 2 * (s2 / vec) + 16 <= 44 * 1024;
            // (forced, any item will do; by default only items worth a block)
            const bool worth = tune.box >= 2 ? std::min(s1, s2) * cnt >= 128
                                             : std::min(s1, s2) * cnt >= 256 && sup * cnt * rpi >= kItemBytes / 4;
            // default policy: where the row, unit or gather walk would run on runs below 256 bytes, and where
            // the zip kernels would zip a digit of fewer than 8 rows or work on short target ranges
            // (measured on the odd-shape sweep: against the unit walk and the gather walk 1.5-1.7x; against the
            // zip kernels 1.1-1.5x where their target ranges are below 768 bytes -- each range pays for its own
            // ragged head and tail --, 1.03-1.06x up to 1536 bytes unless the fan-out is 8 or more, 1.04-1.15x
            // where the zipped digit has fewer than 8 rows, 0.97x elsewhere)
            const i64 zip_range = zip_n * (m2[kp] > 1 ? std::max(m1[kp], m2[kp]) * run_bytes : run_bytes);
            // Two more cases go to the super-boxes, found by probing row-to-column transposes over 8-64 tiles:
            // zip launches that could use neither the periodic nor the by-range walk (tabulated or flat walk:
            // 0.88x of the super-boxes on 33 problems of the sweep, 2.8-3.0 against 4.1-5.2 TB/s on 2-byte units),
            // and long source rows of runs up to 16 bytes unzipped into 16 or more tiles, where every store
            // instruction of the zip walk scatters 16-byte pieces over as many tiles (32 and 64 tiles: 2.3-2.8
            // against 4.5-5.8 TB/s; 16 tiles: 4.3-4.6 against 5.6-6.1 on 12- and 14-byte runs, 4.8 against 4.4 on 6-byte runs).
            bool zip_slow = false;
            if (zip_n > 0) {
                const bool ld = m2[kp] > 1;
                const i64 zm = std::max(m1[kp], m2[kp]), row_bytes = zm * run_bytes;
                const i64 zseg = ld ? zm : 1, seg_row = ld ? run_bytes : row_bytes;
                i64 rpb = std::max<i64>(1, std::min<i64>(zip_n, kItemBytes / row_bytes));
                rpb = std::max<i64>(1, std::min<i64>(rpb, (38 * 1024 / zseg - 48) / seg_row));
                const i64 L = ld ? row_bytes : run_bytes, pc = L / std::gcd<i64>(16, L);
                const i64 lanes_needed = !ld && run_bytes <= 16 ? pc * zm : pc;
                const bool periodic = (tune.zip_walks & 1) && lanes_needed <= kBlockThreads - 1 && rpb * L / 16 >= 2 * pc;
                const bool by_range = (tune.zip_walks & 2) && run_bytes * 4 >= 32 * vec && vec < 16 &&
                                      rpb * (ld ? zm : 1) * ((run_bytes + 15) / 16) >= std::max<i64>(1, tune.zip_by_range_slots);
                zip_slow = (!periodic && !by_range) || (!ld && run_bytes <= 16 && zm >= 16);
            }
            const bool wanted = tune.box >= 2 ||
                                (zip_n > 0 ? (zip_range < 1536 && (zip_range < 768 || fan < 8)) || zip_n < 8 || zip_slow
                                           : run_bytes < 256);
            if (!fits || !worth || !wanted || sup > (1ll << 30)) bxK = -2;
        }
    }
    if (bxK >= -1) {
        // unit digits from scratch: boxes of g for the dimensions up to K, super-boxes for the inner ones
        n_boxes = 1;
        nu = 0;
        size_t bi = 0;
        for (int k = 0; k < r; ++k) {
            const bool in = k >= bxd.front().k && k <= kp;
            const i64 mul = in ? bxd[bi].E / g[k] : 1;
            if (in) ++bi;
            if (nq[k] == 1) continue;
            G.unit_n[nu] = make_div(uint32_t(nq[k] / mul));
            G.unit_mul[nu] = uint32_t(mul);
            G.unit_m1[nu] = make_div(uint32_t(m1[k]));
            G.unit_m2[nu] = make_div(uint32_t(m2[k]));
            G.unit_ts1[nu] = uint32_t(ts1[k]);
            G.unit_ts2[nu] = uint32_t(ts2[k]);
            G.unit_b1[nu] = g[k] * es1[k] * e;
            G.unit_b2[nu] = g[k] * es2[k] * e;
            n_boxes *= nq[k] / mul;
            ++nu;
        }
        G.n_unit = nu;
        G.inner_n = make_div(1);
        G.inner_digit = 0xffffffffu;
        G.inner_span = 1;
        G.inner_mul = 1;
        inner = 1;
        G.fast_boxes = make_div(1);
        // row digits: the dimensions before K (merged where both sides stay contiguous), K itself, then the
        // inner dimensions but the last as plain row digits of a box (the kernel does not use those: it
        // works on the super-box, whose rows are described by the bx_ fields)
        rows.clear();
        for (int k = 0; k < bxK; ++k)
            if (g[k] > 1) rows.push_back(RowDigit{g[k], es1[k] * e, es2[k] * e});
        for (size_t q = rows.size(); q-- > 1;) {
            RowDigit &o = rows[q - 1], &in = rows[q];
            if (o.b1 == in.n * in.b1 && o.b2 == in.n * in.b2) {
                in.n *= o.n;
                rows.erase(rows.begin() + (q - 1));
            }
        }
        const size_t n_outer = rows.size();
        i64 tab_rows = 1;
        for (const RowDigit &d : rows) tab_rows *= d.n;
        rows.push_back(RowDigit{bx_gK, bxK >= 0 ? es1[bxK] * e : 0, bxK >= 0 ? es2[bxK] * e : 0});
        for (size_t q = 0; q + 1 < bxd.size(); ++q)
            if (g[bxd[q].k] > 1) rows.push_back(RowDigit{g[bxd[q].k], es1[bxd[q].k] * e, es2[bxd[q].k] * e});
        if (rows.size() > size_t(kMaxRowDigits)) return REDIST_EUNSUPPORTED;
        n_rows = 1;
        for (size_t q = 0; q < rows.size(); ++q) {
            G.row_n[q] = make_div(uint32_t(rows[q].n));
            G.row_b1[q] = rows[q].b1;
            G.row_b2[q] = rows[q].b2;
            n_rows *= rows[q].n;
        }
        G.n_row = uint32_t(rows.size());
        G.mode = kModeBox;
        G.rows = uint32_t(tab_rows);
        G.n_row_tab = uint32_t(n_outer);
        G.tab_inner = make_div(uint32_t(bx_gK));
        G.units_per_run = make_div(uint32_t(run_bytes / vec));
        G.rows_per_item = uint32_t(bx_rpi);
        G.per_block = uint32_t(bx_cnt);
        const i64 ncb = (bx_gK + bx_cnt - 1) / bx_cnt;
        G.col_blocks = make_div(uint32_t(ncb));
        i64 trail = e;
        for (int k = kp + 1; k < r; ++k) trail *= a.tile[k];
        i64 n1 = 1, n2 = 1;
        G.bx_n = uint32_t(bxd.size());
        // The innermost digit of a position inside a target row is the unit inside a run (the run is
        // contiguous on both sides, and the unit size divides it but not necessarily the trailing
        // dimensions); the last inner dimension therefore counts runs: its extents are divided by the gcd.
        const i64 gl = g[kp];
        for (size_t q = bxd.size(); q-- > 0;) {
            // inner to outer: strides inside a source segment row, segment steps
            i64 st = run_bytes, seg = 1;
            for (size_t w = q + 1; w < bxd.size(); ++w) {
                st *= bxd[w].c1 / (w + 1 == bxd.size() ? gl : 1);
                seg *= bxd[w].E / bxd[w].c1;
            }
            const i64 sc = q + 1 == bxd.size() ? gl : 1;
            G.bx_c1[q] = make_div(uint32_t(bxd[q].c1 / sc));
            G.bx_c2[q] = make_div(uint32_t(bxd[q].c2 / sc));
            G.bx_n1[q] = make_div(uint32_t(bxd[q].E / bxd[q].c1));
            G.bx_n2[q] = make_div(uint32_t(bxd[q].E / bxd[q].c2));
            G.bx_ts1[q] = uint32_t(ts1[bxd[q].k]);
            G.bx_ts2[q] = uint32_t(ts2[bxd[q].k]);
            G.bx_st1[q] = uint32_t(st);
            G.bx_seg[q] = uint32_t(seg);
            n1 *= bxd[q].E / bxd[q].c1;
            n2 *= bxd[q].E / bxd[q].c2;
        }
        G.bx_trail = make_div(uint32_t(run_bytes / vec));
        G.bx_s1 = uint32_t(bx_s1);
        G.bx_s2 = make_div(uint32_t(bx_s2));
        G.bx_nseg = uint32_t(n1);
        G.bx_nrng = uint32_t(n2);
        G.bx_nseg_div = make_div(uint32_t(n1));
        G.bx_nrng_div = make_div(uint32_t(n2));
        G.zip_seg_pitch = uint32_t(round_up(bx_cnt * bx_s1, 16) + 32);
        G.stage_pitch = uint32_t(G.zip_seg_pitch * n1);          // one outer row of the item
        G.zip_lut_units = uint32_t(bx_s2 / vec);
        G.bx_row_units_div = make_div(uint32_t(bx_s2 / vec));
        G.zip_slots = make_div(uint32_t(bx_cnt * bx_s2 / 16 + 1));
        {
            // Lanes per range (a power of two; groups of that many lanes share out the ranges of the item).
            // Two things decide: how evenly ranges and chunks divide among the groups, and the shared-memory
            // banks.  Where the units of one target tile sit a power-of-two stride apart in the staged
            // segments (a tile that takes one element in 4 or 8 of the last dimension), the lanes of a warp
            // that all work on one range read from 1-4 of the 32 banks; neighbouring ranges start a few
            // bytes apart, so narrower groups -- several ranges per warp -- spread the reads.  For every
            // width the banks of the first warp's reads are counted and the time of the item estimated as
            //     (warp, step) pairs with a lane at work  x  (52 issue slots + wavefronts of the reads)
            //                                             x  (1 + 4 / warps that have work)
            // (constants fitted to the measured times of 119 launches at seven widths each; choosing by the
            // estimate is within 0.3 % of choosing by the measurement, geometric mean, 3.6 % at worst).
            const i64 chunks = bx_cnt * bx_s2 / 16, ranges = bx_rpi * n2;
            const uint32_t unit = uint32_t(vec), per = 16u / unit;
            auto place = [&](uint32_t p) {
                uint32_t rest = p / G.bx_trail.d, off = (p % G.bx_trail.d) * unit;
                for (int q = int(G.bx_n) - 1; q >= 0; --q) {
                    const uint32_t i = rest % G.bx_c2[q].d;
                    rest /= G.bx_c2[q].d;
                    off += i / G.bx_c1[q].d * G.bx_seg[q] * G.zip_seg_pitch + i % G.bx_c1[q].d * G.bx_st1[q];
                }
                return off;
            };
            auto base = [&](uint32_t range) {
                uint32_t rem = range % uint32_t(n2), off = range / uint32_t(n2) * G.stage_pitch;
                for (int q = int(G.bx_n) - 1; q >= 0; --q) {
                    const uint32_t x = rem % G.bx_n2[q].d * G.bx_c2[q].d;
                    rem /= G.bx_n2[q].d;
                    off += x / G.bx_c1[q].d * G.bx_seg[q] * G.zip_seg_pitch + x % G.bx_c1[q].d * G.bx_st1[q];
                }
                return off;
            };
            const uint32_t row_units = G.zip_lut_units;
            auto wavefronts = [&](i64 width) {                 // of the first warp's reads of one chunk each
                const uint32_t phase_lanes = std::min(32u, 32u * 4u / unit);   // 8- and 16-byte reads go in half and quarter warps
                uint32_t total = 0;
                for (uint32_t i = 0; i < per; ++i)
                    for (uint32_t l0 = 0; l0 < 32u; l0 += phase_lanes) {
                        uint32_t words[32][32], n_words[32] = {0}, worst = 0;
                        for (uint32_t l = l0; l < l0 + phase_lanes; ++l) {
                            const uint32_t range = l / uint32_t(width), c = l % uint32_t(width);
                            if (i64(range) >= ranges || i64(c) >= chunks) continue;
                            const uint32_t x = c * per + i;
                            const uint32_t at = base(range) + x / row_units * G.bx_s1 + place(x % row_units);
                            for (uint32_t b = 0; b < std::max(1u, unit / 4u); ++b) {
                                const uint32_t word = at / 4u + b, bank = word & 31u;
                                bool seen = false;
                                for (uint32_t k = 0; k < n_words[bank]; ++k) seen |= words[bank][k] == word;
                                if (!seen) words[bank][n_words[bank]++] = word;
                                worst = std::max(worst, n_words[bank]);
                            }
                        }
                        total += worst;
                    }
                return total;
            };
            auto estimate = [&](i64 width) {
                const i64 groups = kBlockThreads / width, steps = (chunks + width - 1) / width;
                auto ranges_of = [&](i64 group) { return group < ranges ? (ranges - group + groups - 1) / groups : 0; };
                i64 pairs = 0, busy = 0;
                if (width >= 32) {
                    for (i64 gi = 0; gi < groups; ++gi) pairs += ranges_of(gi) * steps * (width / 32);
                    busy = std::min<i64>(kBlockThreads / 32, std::min(groups, ranges) * (width / 32));
                } else {
                    const i64 per_warp = 32 / width;
                    for (i64 v = 0; v < kBlockThreads / 32; ++v) {
                        const i64 most = ranges_of(v * per_warp);   // the first group of a warp has the most ranges
                        pairs += most * steps;
                        busy += most > 0;
                    }
                }
                return double(pairs) * double(52 + wavefronts(width)) * (1.0 + 4.0 / double(std::max<i64>(1, busy)));
            };
            i64 best = 2;
            double best_cost = estimate(2);
            for (i64 cand = 4; cand <= 128; cand *= 2) {
                const double cost = estimate(cand);
                if (cost < best_cost * 0.999) {
                    best = cand;
                    best_cost = cost;
                }
            }
            if (tune.box_width > 0 && (tune.box_width & (tune.box_width - 1)) == 0) best = tune.box_width;
            G.zip_width = uint32_t(best);
        }
        G.gl_m = make_div(1);
        ipb = (tab_rows + bx_rpi - 1) / bx_rpi * ncb;
    } else if (zip_n > 0) {
        const bool long_dst = m2[kp] > 1;
        const i64 m = std::max(m1[kp], m2[kp]);
        const i64 nseg = long_dst ? m : 1;                 // source segments per table row
        const i64 row_bytes = m * run_bytes;               // both sides, per row of the zipped digit
        const i64 tab_rows = n_rows / zip_n;
        const i64 seg_row = long_dst ? run_bytes : row_bytes;   // bytes of one row in a source segment
        const i64 kTile = 38 * 1024;                            // shared-memory tile of an item, at most
        const i64 kZipBytes = kItemBytes;
        i64 rpb = std::max<i64>(1, std::min<i64>(zip_n, kZipBytes / row_bytes));
        rpb = std::max<i64>(1, std::min<i64>(rpb, (kTile / nseg - 48) / seg_row));
        const i64 ncb = (zip_n + rpb - 1) / rpb;
        const i64 seg_pitch = round_up(rpb * seg_row, 16) + 32;
        i64 rpi = std::max<i64>(1, kZipBytes / (rpb * row_bytes));
        rpi = std::min<i64>(std::min<i64>(rpi, tab_rows), std::max<i64>(1, kZipSegments / nseg));
        rpi = std::max<i64>(1, std::min<i64>(rpi, kTile / (seg_pitch * nseg)));
        if (seg_pitch * nseg * rpi > kTile) return REDIST_EINTERNAL;
        G.mode = kModeZip;
        G.gl_levels = 0;
        G.gl_stretch = 0;
        G.gl_m = make_div(uint32_t(m));
        G.inner_mul = uint32_t(m);
        G.inner_n = make_div(1);
        inner = 1;
        G.gl_long_dst = long_dst ? 1u : 0u;
        G.gl_ts = long_dst ? G.unit_ts1[G.inner_digit] : G.unit_ts2[G.inner_digit];
        G.rows = uint32_t(tab_rows);
        G.n_row_tab = uint32_t(rows.size() - 1);
        G.tab_inner = make_div(uint32_t(zip_n));
        G.units_per_run = make_div(uint32_t(run_bytes / vec));
        G.rows_per_item = uint32_t(rpi);
        G.per_block = uint32_t(rpb);
        G.col_blocks = make_div(uint32_t(ncb));
        G.zip_seg_pitch = uint32_t(seg_pitch);
        G.zip_tile_fastest = !long_dst && run_bytes <= 16 ? 1u : 0u;
        G.stage_pitch = uint32_t(seg_pitch * nseg);
        {
            // periodic walk: a table row must give every thread several chunks, and the period must leave most
            // threads of a block busy
            const i64 kZipPeriodic = (tune.zip_walks & 1) ? 1 : 0;
            const i64 L = long_dst ? row_bytes : run_bytes;         // bytes after which the target pattern repeats, up to alignment
            const i64 gc = std::gcd<i64>(16, L);
            const i64 pc = L / gc;
            G.zip_period = FastDiv{0, 0, 0};
            G.zip_period_rows = 0;
            G.zip_width = 0;
            // longest period, in chunks (the lanes of one block must span it; above 128 the launch uses 256 threads)
            const i64 kZipPc = kBlockThreads - 1;
            // (with long source rows of runs up to 16 bytes a thread stays with one of the m target tiles)
            const i64 lanes_needed = !long_dst && run_bytes <= 16 ? pc * m : pc;
            const i64 range_chunks = rpb * L / 16;                  // chunks of one target range, at most
            if (kZipPeriodic > 0 && rpb * row_bytes / 16 >= kZipPeriodic && lanes_needed <= kZipPc && range_chunks >= 2 * pc) {
                G.zip_period = make_div(uint32_t(pc));
                G.zip_period_rows = uint32_t(16 / gc);
                // lanes per table row: about kZipLaneChunks chunks of a range for each, so that the decode of a
                // lane's first chunk is shared by several chunks while short ranges still fill the block
                const i64 kZipLaneChunks = 4;
                const i64 want = std::max<i64>(1, (range_chunks + kZipLaneChunks * pc - 1) / (kZipLaneChunks * pc));
                G.zip_width = uint32_t(std::min<i64>(want * pc, kBlockThreads / pc * pc));
            }
        }
        // By-range walk: for runs of eight units and more (32 bytes of 4-byte units, 64 of 8-byte units; nothing
        // to gain with 16-byte units) the chunk slots of a range are numbered (run, i-th target-aligned chunk
        // that starts in the run) -- such a chunk takes its units from that run and, past its end, from the
        // next one, no division per unit -- and a range with 256 slots or more is walked by the whole block.
        const i64 kZipPerRun = (tune.zip_walks & 2) ? 32 : 0;   // shortest run (of 4-byte units) for the by-range walk
        const i64 kZipByRange = std::max<i64>(1, tune.zip_by_range_slots);
        const i64 cpr = (run_bytes + 15) / 16;
        if (G.zip_period.d == 0 && kZipPerRun > 0 && run_bytes * 4 >= kZipPerRun * vec && vec < 16 &&
            rpb * (long_dst ? m : 1) * cpr >= kZipByRange) {
            G.zip_cpr = make_div(uint32_t(cpr));
            G.zip_slots = make_div(uint32_t(rpb * (long_dst ? m : 1) * cpr));
        } else {
            G.zip_cpr = FastDiv{0, 0, 0};
            G.zip_slots = make_div(uint32_t(rpb * (long_dst ? row_bytes : run_bytes) / 16 + 1));
        }
        {
            // short ranges (neither walk above applies): the place of every unit of a range is tabulated in shared
            // memory; the chunk slots are then numbered flat
            const i64 kZipLut = (tune.zip_walks & 4) ? 2048 : 0;   // longest range, in units, whose unit places are tabulated
            const i64 units = rpb * (long_dst ? row_bytes : run_bytes) / vec;
            G.zip_lut_units = 0;
            if (G.zip_period.d == 0 && G.zip_cpr.d == 0 && units <= kZipLut && seg_pitch * nseg * rpi + units * 4 <= 42 * 1024)
                G.zip_lut_units = uint32_t(units);
        }
        ipb = (tab_rows + rpi - 1) / rpi * ncb;
    } else if (g_levels >= 0) {
        const bool long_dst = m2[kp] > 1;
        const i64 m = std::max(m1[kp], m2[kp]);
        i64 tab_inner = 1;
        for (int l = 0; l < g_levels; ++l) {
            const RowDigit &d = rows[rows.size() - 1 - size_t(l)];
            G.gl_n[l] = make_div(uint32_t(d.n));
            G.gl_b1[l] = d.b1;
            tab_inner *= d.n;
        }
        const i64 tab_rows = n_rows / tab_inner;
        const i64 ns = long_dst ? 1 : m;                  // stretches per table row
        const i64 per_row = g_stretch / 16;
        const i64 cpb = std::max<i64>(1, std::min<i64>(per_row, kItemBytes / 16));
        const i64 ncb = std::max<i64>(1, (per_row + cpb - 1) / cpb);
        i64 rpi = std::max<i64>(1, std::min<i64>(kMaxRowsFlat, kItemBytes / (cpb * 16 * ns)));
        rpi = std::min<i64>(rpi, tab_rows);
        G.mode = kModeGather;
        G.gl_levels = uint32_t(g_levels);
        G.gl_stretch = uint32_t(g_stretch);
        G.gl_m = make_div(uint32_t(m));
        G.inner_mul = uint32_t(m);
        G.inner_n = make_div(1);
        inner = 1;
        G.gl_long_dst = long_dst ? 1u : 0u;
        G.gl_ts = long_dst ? G.unit_ts1[G.inner_digit] : G.unit_ts2[G.inner_digit];
        G.rows = uint32_t(tab_rows);
        G.n_row_tab = uint32_t(rows.size() - size_t(g_levels));
        G.tab_inner = make_div(uint32_t(tab_inner));
        G.units_per_run = make_div(uint32_t(run_bytes / vec));
        G.rows_per_item = uint32_t(rpi);
        G.per_block = uint32_t(cpb);
        G.col_blocks = make_div(uint32_t(ncb));
        ipb = (tab_rows + rpi - 1) / rpi * ncb;
    } else if (G.aligned && max_chunks <= kBlockThreads) {
        // aligned short runs: `lanes` threads per row, one chunk each
        const i64 kItemBytes = bulk_item_bytes;
        const i64 lanes = max_chunks;
        G.mode = kModeRows;
        G.lanes = uint32_t(lanes);
        G.rows_per_pass = uint32_t(kBlockThreads / lanes);
        i64 rpi = std::max<i64>(G.rows_per_pass, kItemBytes / run_bytes / G.rows_per_pass * G.rows_per_pass);
        rpi = std::min<i64>(rpi, round_up(n_rows, G.rows_per_pass));
        G.rows_per_item = uint32_t(rpi);
        G.per_block = uint32_t(max_chunks);
        G.col_blocks = make_div(1);
        ipb = (n_rows + rpi - 1) / rpi;
    } else {
        // flat walk over (row, chunk) -- or, for short ragged runs, over (table row, unit piece) where a
        // table row carries all the runs of the innermost row digit
        const i64 kItemBytes = bulk_item_bytes;
        const bool units = run_bytes < 256;
        i64 tab_inner = 1, tab_rows = n_rows;
        if (units && run_bytes <= 16 && !rows.empty() && rows.back().n * (run_bytes / vec) < (1ll << 30)) {
            // only when a table of rows could not fill an item (and the payload index fits 32 bits)
            tab_inner = rows.back().n;
            tab_rows = n_rows / tab_inner;
        }
        const i64 per_row = units ? tab_inner * (run_bytes / vec) : max_chunks;
        const i64 piece = units ? vec : 16;
        const i64 cpb = std::max<i64>(1, std::min<i64>(per_row, kItemBytes / piece));
        const i64 ncb = std::max<i64>(1, (per_row + cpb - 1) / cpb);
        i64 rpi = std::max<i64>(1, std::min<i64>(kMaxRowsFlat, kItemBytes / (cpb * piece)));
        rpi = std::min<i64>(rpi, tab_rows);
        if (!units && !G.aligned && kBulk) {
            // ragged rows: each row segment is loaded by one bulk copy of the 16-byte blocks that cover
            // it (up to 15 bytes before and after, plus the ragged head), then shifted out of shared memory
            const i64 pitch = cpb * 16 + 64;
            const i64 kRaggedKb = 38;      // shared-memory tile of a ragged bulk item, KiB
            rpi = std::max<i64>(1, std::min<i64>(rpi, std::min<i64>(kRaggedBulkRows, kRaggedKb * 1024 / pitch)));
            ragged_bulk = true;
            G.stage_pitch = uint32_t(pitch);
            // lanes that walk one row together: about four chunks each, a whole number of warps
            // (and no more groups than rows)
            i64 w = 32;
            while (w < kBlockThreads && (w * 4 < cpb || (kBlockThreads / w) > rpi)) w *= 2;
            G.lanes = uint32_t(w);
        }
        G.mode = units ? kModeUnits : kModeChunks;
        G.rows = uint32_t(tab_rows);
        G.n_row_tab = uint32_t(tab_inner > 1 ? rows.size() - 1 : rows.size());
        G.tab_inner = make_div(uint32_t(tab_inner));
        G.units_per_run = make_div(uint32_t(std::max<i64>(1, run_bytes / vec)));
        G.rows_per_item = uint32_t(rpi);
        G.per_block = uint32_t(cpb);
        G.col_blocks = make_div(uint32_t(ncb));
        ipb = (tab_rows + rpi - 1) / rpi * ncb;
    }
    G.bulk = ragged_bulk ? 2u : 0u;
    if (kBulk && G.aligned && (G.mode == kModeRows || G.mode == kModeChunks)) {
        const i64 seg = G.mode == kModeRows ? run_bytes : i64(G.per_block) * 16;
        if (seg >= kBulkMin && G.rows_per_item <= uint32_t(kBulkThreads) && seg * G.rows_per_item <= 47 * 1024) G.bulk = 1;
    }
    G.per_block_div = make_div(G.per_block);
    G.lanes_div = make_div(G.lanes);
    if (ipb >= (1ll << 31) || n_boxes * ipb * inner >= (1ll << 31)) return REDIST_EUNSUPPORTED;
    G.items_per_box = make_div(uint32_t(ipb));
    G.n_items = uint32_t(n_boxes * ipb * inner);

    // tables
    i64 nt1 = 1, nt2 = 1;
    for (int k = 0; k < r; ++k) {
        nt1 *= a.ntiles[k];
        nt2 *= b.ntiles[k];
    }
    const int N = p.n_devices;
    out.src_holder.assign(size_t(nt1), -1);
    out.src_tile_of.assign(size_t(N), -1);
    if (!a.shared_global) {
        for (int d = 0; d < N; ++d) out.src_tile_of[d] = a.tile_of[d];
        for (int d = N - 1; d >= 0; --d) out.src_holder[a.tile_of[d]] = d;   // lowest id holding the tile
        for (int32_t h : out.src_holder)
            if (h < 0) return REDIST_EINTERNAL;
    }
    if (b.shared_global) {
        G.fanout = 1;
        out.dst_devs.assign(1, -1);
    } else {
        if (N % nt2) return REDIST_EINTERNAL;
        const i64 R = N / nt2;
        G.fanout = uint32_t(R);
        out.dst_devs.assign(size_t(nt2 * R), -1);
        std::vector<int> fill(size_t(nt2), 0);
        for (int d = 0; d < N; ++d) {
            int32_t t = b.tile_of[d];
            if (fill[t] >= R) return REDIST_EINTERNAL;
            out.dst_devs[size_t(t) * R + fill[t]++] = d;
        }
    }
    i64 gsize = 1, l1 = 1, l2 = 1;
    for (int k = 0; k < r; ++k) {
        gsize *= p.global_shape[k];
        l1 *= a.tile[k];
        l2 *= b.tile[k];
    }
    G.wait_polls = uint32_t(std::max<i64>(1, std::min<i64>(tune.wait_polls, 1ll << 30)));
    // evict-first stores measured on the plain bulk-copy kernels by fan-out: 1: +0.1 %, 2: -0.4 %, 4: +0.5 %, 8 and
    // 16: +1.1 % (c3c 6.50 -> 6.55 TB/s); evict-first loads cost 0.6-1.7 % everywhere
    G.l2_hint = tune.l2_hint == 4 ? (fan >= 4 ? 2u : 0u) : uint32_t(tune.l2_hint);
    // super-boxes of 1- and 2-byte units on runs of 64 bytes and more: most chunks lie inside one run, and the kernel
    // that reads such a chunk as one unaligned 16-byte piece pays (1.2-1.3x on 1-byte units, 1.0-1.1x on 2-byte
    // units; 0.85x on runs below 64 bytes; in the zip kernels 0.93-0.98x, not built)
    G.one_piece = tune.piece != 0 && vec < 4 && run_bytes >= 64 && G.mode == kModeBox ? 1u : 0u;
    G.test_extra_tx = uint32_t(std::max<i64>(0, std::min<i64>(tune.test_extra_tx, 1 << 20)));
    G.n_src_tab = uint32_t(out.src_holder.size());
    G.n_dst_tab = uint32_t(out.dst_devs.size());
    // (test_shrink_tiles, test only: the checked build is told shorter tiles, so that the last accesses of
    // every tile fail their test, are skipped and are counted -- the positive control of that build)
    G.src_tile_bytes = uint64_t(std::max<i64>(0, l1 * e - tune.test_shrink_tiles));
    G.dst_tile_bytes = uint64_t(std::max<i64>(0, l2 * e - tune.test_shrink_tiles));
    out.run_bytes = run_bytes;
    out.src_tile = a.tile;
    out.dst_tile = b.tile;
    out.src_tile_bytes = l1 * e;
    out.dst_tile_bytes = l2 * e;
    out.bytes_read = gsize * e;
    out.bytes_written = b.shared_global ? gsize * e : i64(N) * l2 * e;
    return REDIST_OK;
}

redist_status build_launches(Plan &p)
{
    const int mode = int(p.flags & REDIST_MODE_MASK);
    const int n = int(p.steps.size());
    const i64 e = p.elem_bytes;
    std::vector<Layout> lay;
    lay.push_back(layout_of(p, p.initial));
    for (const Step &s : p.steps) lay.push_back(layout_of(p, s.post));
    p.launches.clear();
    p.slot_bytes = 0;
    i64 gsize = 1;
    for (i64 s : p.global_shape) gsize *= s;

    auto add = [&](int s0, int s1, int kernel) -> redist_status {
        Launch L;
        L.first_step = s0;
        L.n_steps = s1 - s0;
        L.kernel = kernel;
        redist_status rc = build_copy(p, lay[s0], lay[s1], L);
        if (rc != REDIST_OK) return rc;
        p.launches.push_back(L);
        return REDIST_OK;
    };

    if (mode == REDIST_NAIVE) {
        Layout glob;
        glob.tile = p.global_shape;
        glob.ntiles.assign(p.rank, 1);
        glob.tile_of.assign(p.n_devices, 0);
        glob.shared_global = true;
        Launch a, b;
        a.first_step = 0; a.n_steps = n; a.kernel = 6;
        b.first_step = 0; b.n_steps = n; b.kernel = 7;
        redist_status rc = build_copy(p, lay.front(), glob, a);
        if (rc == REDIST_OK) rc = build_copy(p, glob, lay.back(), b);
        if (rc != REDIST_OK) return rc;
        a.from = BUF_SRC; a.to = BUF_GLOBAL;
        b.from = BUF_GLOBAL; b.to = BUF_DST;
        p.launches = {a, b};
        p.scratch_bytes = round_up(gsize * e, 256);
        p.scratch_per_device = gsize * e;
    } else {
        std::vector<std::pair<int, int>> segs;
        if (n == 0 || mode == REDIST_FUSE_ALL) {
            segs.push_back({0, n});
        } else if (mode == REDIST_FUSE_NONE) {
            for (int s = 0; s < n; ++s) segs.push_back({s, s + 1});
        } else {
            // fuse adjacent steps while the fused copy keeps runs of 64 bytes, or at least as long
            // as the shortest run of the steps it replaces
            int s = 0;
            while (s < n) {
                int t = s + 1;
                Launch probe;
                redist_status rc = build_copy(p, lay[s], lay[t], probe);
                if (rc != REDIST_OK) return rc;
                i64 min_run = probe.run_bytes;
                while (t < n) {
                    Launch one, fused;
                    rc = build_copy(p, lay[t], lay[t + 1], one);
                    if (rc == REDIST_OK) rc = build_copy(p, lay[s], lay[t + 1], fused);
                    if (rc != REDIST_OK) return rc;
                    i64 mr = std::min(min_run, one.run_bytes);
                    if (fused.run_bytes < 64 && fused.run_bytes < mr) break;
                    min_run = mr;
                    ++t;
                }
                segs.push_back({s, t});
                s = t;
            }
        }
        for (auto &sg : segs) {
            int kernel = 5;
            if (sg.second - sg.first == 0) kernel = REDIST_STEP_COPY;
            if (sg.second - sg.first == 1) kernel = p.steps[sg.first].kind;
            redist_status rc = add(sg.first, sg.second, kernel);
            if (rc != REDIST_OK) return rc;
        }
        const int nl = int(p.launches.size());
        i64 slot = 0;
        for (int q = 0; q + 1 < nl; ++q) slot = std::max(slot, p.launches[q].dst_tile_bytes);
        p.slot_bytes = round_up(slot, 256);
        const int nslots = nl <= 1 ? 0 : (nl == 2 ? 1 : 2);
        for (int q = 0; q < nl; ++q) {
            p.launches[q].from = q == 0 ? BUF_SRC : ((q - 1) % 2 ? BUF_SCRATCH1 : BUF_SCRATCH0);
            p.launches[q].to = q == nl - 1 ? BUF_DST : (q % 2 ? BUF_SCRATCH1 : BUF_SCRATCH0);
        }
        p.scratch_per_device = nslots * p.slot_bytes;
        p.scratch_bytes = p.scratch_per_device * p.n_devices;
    }
    p.alignment = 16;   // every tile and scratch pointer; offsets inside a tile may be finer
    return REDIST_OK;
}

}  // namespace redist
