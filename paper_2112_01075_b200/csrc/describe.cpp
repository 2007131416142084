// JSON description of a plan: the typed sequence with its device maps, and the launch descriptors.
#include <sstream>

#include "plan.hpp"

namespace redist {

namespace {

template <class T>
void arr(std::ostringstream &o, const std::vector<T> &v)
{
    o << "[";
    for (size_t i = 0; i < v.size(); ++i) o << (i ? "," : "") << (long long)v[i];
    o << "]";
}

template <class T>
void arr2(std::ostringstream &o, const std::vector<std::vector<T>> &v)
{
    o << "[";
    for (size_t i = 0; i < v.size(); ++i) {
        if (i) o << ",";
        arr(o, v[i]);
    }
    o << "]";
}

void state(std::ostringstream &o, const char *name, const ConcreteState &s)
{
    o << "\"" << name << "_axes\":";
    arr2(o, s.ax);
    o << ",\"" << name << "_coords\":";
    arr2(o, s.lc);
}

void fd(std::ostringstream &o, const FastDiv *f, uint32_t n)
{
    o << "[";
    for (uint32_t i = 0; i < n; ++i) o << (i ? "," : "") << f[i].d;
    o << "]";
}

template <class T>
void raw(std::ostringstream &o, const T *v, uint32_t n)
{
    o << "[";
    for (uint32_t i = 0; i < n; ++i) o << (i ? "," : "") << (long long)v[i];
    o << "]";
}

const char *kKind[] = {"dynslice", "alltoall", "allgather", "allpermute", "copy"};
const char *kKernel[] = {"dynslice", "alltoall", "allgather", "allpermute", "copy", "fused", "naive_gather", "naive_slice"};
const char *kBuf[] = {"src", "dst", "scratch0", "scratch1", "global"};

}  // namespace

void describe(Plan &p)
{
    std::ostringstream o;
    o << "{\"mesh_shape\":";
    arr(o, p.mesh_shape);
    o << ",\"global_shape\":";
    arr(o, p.global_shape);
    o << ",\"elem_bytes\":" << p.elem_bytes << ",\"n_devices\":" << p.n_devices << ",\"flags\":" << p.flags;
    o << ",\"primes\":[";
    for (size_t a = 0; a < p.primes.size(); ++a)
        o << (a ? "," : "") << "{\"parent\":" << p.primes[a].parent << ",\"size\":" << p.primes[a].size
          << ",\"stride\":" << p.primes[a].parent_stride << "}";
    o << "],\"src_axes\":";
    arr2(o, p.src_pax);
    o << ",\"dst_axes\":";
    arr2(o, p.dst_pax);
    o << ",\"initial_coords\":";
    arr2(o, p.initial.lc);
    o << ",\"local_src\":" << p.local_src << ",\"local_dst\":" << p.local_dst << ",\"height\":" << p.height
      << ",\"cost\":" << p.cost << ",\"slot_bytes\":" << p.slot_bytes << ",\"scratch_bytes\":" << p.scratch_bytes
      << ",\"scratch_per_device\":" << p.scratch_per_device << ",\"alignment\":" << p.alignment;
    o << ",\"steps\":[";
    for (size_t s = 0; s < p.steps.size(); ++s) {
        const Step &st = p.steps[s];
        o << (s ? "," : "") << "{\"kind\":\"" << kKind[st.kind] << "\",\"i\":" << st.dim_i << ",\"j\":" << st.dim_j
          << ",\"factor\":" << st.factor << ",\"acting\":";
        arr(o, st.acting);
        o << ",";
        state(o, "pre", st.pre);
        o << ",";
        state(o, "post", st.post);
        o << ",\"source_of\":";
        arr(o, st.source_of);
        o << ",\"local_before\":";
        arr(o, st.local_before);
        o << ",\"local_after\":";
        arr(o, st.local_after);
        o << ",\"cost\":" << st.cost << "}";
    }
    o << "],\"launches\":[";
    for (size_t l = 0; l < p.launches.size(); ++l) {
        const Launch &L = p.launches[l];
        const CopyGeometry &G = L.geo;
        o << (l ? "," : "") << "{\"first_step\":" << L.first_step << ",\"n_steps\":" << L.n_steps << ",\"kernel\":\""
          << kKernel[L.kernel] << "\",\"from\":\"" << kBuf[L.from] << "\",\"to\":\"" << kBuf[L.to] << "\""
          << ",\"run_bytes\":" << L.run_bytes << ",\"bytes_read\":" << L.bytes_read << ",\"bytes_written\":"
          << L.bytes_written << ",\"src_tile_bytes\":" << L.src_tile_bytes << ",\"dst_tile_bytes\":"
          << L.dst_tile_bytes << ",\"geometry\":{\"fanout\":" << G.fanout << ",\"aligned\":" << G.aligned
          << ",\"unit_bytes\":" << G.unit_bytes << ",\"mode\":" << G.mode << ",\"bulk\":" << G.bulk << ",\"run_bytes\":" << G.run_bytes
          << ",\"per_block\":" << G.per_block << ",\"col_blocks\":" << G.col_blocks.d
          << ",\"lanes\":" << G.lanes << ",\"rows_per_pass\":" << G.rows_per_pass << ",\"rows\":" << G.rows
          << ",\"rows_per_item\":" << G.rows_per_item << ",\"items_per_box\":" << G.items_per_box.d << ",\"fast_boxes\":" << G.fast_boxes.d
          << ",\"n_items\":" << G.n_items << ",\"n_row_tab\":" << G.n_row_tab << ",\"tab_inner\":" << G.tab_inner.d << ",\"inner_n\":" << G.inner_n.d << ",\"inner_digit\":" << int(G.inner_digit) << ",\"inner_span\":" << G.inner_span << ",\"inner_mul\":" << G.inner_mul << ",\"gl_long_dst\":" << G.gl_long_dst << ",\"stage_pitch\":" << G.stage_pitch
          << ",\"units_per_run\":" << G.units_per_run.d << ",\"gl_levels\":" << G.gl_levels << ",\"gl_stretch\":" << G.gl_stretch
          << ",\"gl_m\":" << G.gl_m.d << ",\"zip_seg_pitch\":" << G.zip_seg_pitch << ",\"zip_slots\":" << G.zip_slots.d << ",\"zip_cpr\":" << G.zip_cpr.d << ",\"zip_lut_units\":" << G.zip_lut_units << ",\"zip_period\":" << G.zip_period.d << ",\"zip_period_rows\":" << G.zip_period_rows << ",\"zip_width\":" << G.zip_width << ",\"l2_hint\":" << G.l2_hint << ",\"one_piece\":" << G.one_piece << ",\"gl_n\":";
        fd(o, G.gl_n, G.gl_levels);
        o << ",\"gl_b1\":";
        raw(o, G.gl_b1, G.gl_levels);
        o << ",\"bx_n\":" << G.bx_n << ",\"bx_s1\":" << G.bx_s1 << ",\"bx_s2\":" << G.bx_s2.d << ",\"bx_nseg\":" << G.bx_nseg
          << ",\"bx_nrng\":" << G.bx_nrng << ",\"bx_trail\":" << G.bx_trail.d << ",\"bx_c1\":";
        fd(o, G.bx_c1, G.bx_n);
        o << ",\"bx_c2\":";
        fd(o, G.bx_c2, G.bx_n);
        o << ",\"bx_n1\":";
        fd(o, G.bx_n1, G.bx_n);
        o << ",\"bx_n2\":";
        fd(o, G.bx_n2, G.bx_n);
        o << ",\"bx_ts1\":";
        raw(o, G.bx_ts1, G.bx_n);
        o << ",\"bx_ts2\":";
        raw(o, G.bx_ts2, G.bx_n);
        o << ",\"bx_st1\":";
        raw(o, G.bx_st1, G.bx_n);
        o << ",\"bx_seg\":";
        raw(o, G.bx_seg, G.bx_n);
        o << ",\"unit_mul\":";
        raw(o, G.unit_mul, G.n_unit);
        o << ",\"unit_n\":";
        fd(o, G.unit_n, G.n_unit);
        o << ",\"unit_m1\":";
        fd(o, G.unit_m1, G.n_unit);
        o << ",\"unit_m2\":";
        fd(o, G.unit_m2, G.n_unit);
        o << ",\"unit_ts1\":";
        raw(o, G.unit_ts1, G.n_unit);
        o << ",\"unit_ts2\":";
        raw(o, G.unit_ts2, G.n_unit);
        o << ",\"unit_b1\":";
        raw(o, G.unit_b1, G.n_unit);
        o << ",\"unit_b2\":";
        raw(o, G.unit_b2, G.n_unit);
        o << ",\"row_n\":";
        fd(o, G.row_n, G.n_row);
        o << ",\"row_b1\":";
        raw(o, G.row_b1, G.n_row);
        o << ",\"row_b2\":";
        raw(o, G.row_b2, G.n_row);
        o << "},\"src_holder\":";
        arr(o, L.src_holder);
        o << ",\"dst_devs\":";
        arr(o, L.dst_devs);
        o << "}";
    }
    o << "]}";
    p.json = o.str();
}

}  // namespace redist
