// Host-side C shim over the library's closed-form index arithmetic, so that the CPU tests can
// compare it with the oracle's running-counter walk.  Built by tests/test_host_index.py.
#include "st_index.cuh"
extern "C" {
long long shim_tri_rows(long long d) { return st::tri_rows(d); }
long long shim_tet_rows(long long d) { return st::tet_rows(d); }
long long shim_tri_encode(long long d, long long i, long long j) { return st::tri_encode(d, i, j); }
long long shim_tet_encode(long long d, long long i, long long j, long long k) { return st::tet_encode(d, i, j, k); }
void shim_tri_decode(long long d, long long p, long long *i, long long *j)
{
    int64_t a, b;
    st::tri_decode(d, p, a, b);
    *i = a; *j = b;
}
void shim_tet_decode(long long d, long long q, long long *i, long long *j, long long *k)
{
    int64_t a, b, c;
    st::tet_decode(d, q, a, b, c);
    *i = a; *j = b; *k = c;
}
// decode every position of a triangle / tetrahedron; returns the number of mismatches with
// the lexicographic walk done right here with a running counter
long long shim_check_all_tri(long long d)
{
    long long bad = 0, p = 0;
    for (long long i = 0; i < d; ++i)
        for (long long j = i; j < d; ++j, ++p) {
            int64_t a, b;
            st::tri_decode(d, p, a, b);
            bad += (a != i) || (b != j) || (st::tri_encode(d, i, j) != p);
        }
    return bad + (p != st::tri_rows(d));
}
long long shim_check_all_tet(long long d)
{
    long long bad = 0, q = 0;
    for (long long i = 0; i < d; ++i)
        for (long long j = i; j < d; ++j)
            for (long long k = j; k < d; ++k, ++q) {
                int64_t a, b, c;
                st::tet_decode(d, q, a, b, c);
                bad += (a != i) || (b != j) || (c != k) || (st::tet_encode(d, i, j, k) != q);
            }
    return bad + (q != st::tet_rows(d));
}
long long shim_simp4_rows(long long d) { return st::simp4_rows(d); }
// every position of the 4-simplex against a running counter; returns the number of mismatches
long long shim_check_all_simp4(long long d)
{
    long long bad = 0, s = 0;
    for (long long i = 0; i < d; ++i)
        for (long long j = i; j < d; ++j)
            for (long long k = j; k < d; ++k)
                for (long long l = k; l < d; ++l, ++s) bad += st::simp4_encode(d, i, j, k, l) != s;
    return bad + (s != st::simp4_rows(d));
}
}
