"""GPU parity: the CUDA library (through its C ABI, via the thin binding) against the
CPU oracle on the same seeded inputs.

Bar: max over elements of ‖v_e − v̂_e‖₂/‖v̂_e‖₂ ≤ 1e-12 in fp64 and ≤ 1e-5 in fp32,
v̂ = oracle (for fp32 the oracle widens the fp32 inputs and computes in fp64).
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL64 = 1e-12
TOL32 = 1e-5


@pytest.fixture(scope="module")
def env():
    import torch
    import oracle
    from paper_2604_19906_b200 import build, inputs, ops
    build.build()
    assert torch.cuda.is_available()
    return {"torch": torch, "oracle": oracle, "inputs": inputs, "ops": ops,
            "dev": torch.device("cuda:0")}


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def to_dev(env, a, dtype=None):
    t = env["torch"].from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.to(env["dev"])


def synth_ih(n, E, seed):
    g = rng(seed)
    S, _ = np.linalg.qr(g.standard_normal((n, n)))
    lam = g.uniform(0.1, 2.0, n)
    c = g.uniform(0.5, 1.5, E)
    D = 1.0 / (((lam[:, None, None] + lam[None, :, None]) + lam[None, None, :])[None]
               + c[:, None, None, None])
    u = g.uniform(-1, 1, (E, n, n, n))
    return np.ascontiguousarray(S), D, u


# --------------------------------------------------------------------------- inverse Helmholtz

@pytest.mark.parametrize("n", list(range(1, 17)) + [20, 24])
@pytest.mark.parametrize("E", [1, 2, 3, 5, 37, 301])
def test_inv_helmholtz_f64_small(env, n, E):
    if n >= 20 and E > 37:
        pytest.skip("large n covered at small E")
    S, D, u = synth_ih(n, E, 1000 * n + E)
    want = env["oracle"].inv_helmholtz(S, D, u)
    got = env["ops"].ekl_tpo_inv_helmholtz(to_dev(env, S), to_dev(env, D), to_dev(env, u))
    env["torch"].cuda.synchronize()
    err = env["oracle"].rel_err_per_element(got.cpu().numpy(), want)
    assert err.max() <= TOL64, (n, E, err.max())


@pytest.mark.parametrize("n", [2, 4, 7, 8, 12, 14, 16])
def test_inv_helmholtz_nonorthogonal_S_pins_transposes(env, n):
    """A non-orthogonal, non-symmetric S separates S from Sᵀ in both stages."""
    g = rng(50 + n)
    E = 33
    S = g.standard_normal((n, n)) / np.sqrt(n)
    D = g.uniform(0.1, 1.3, (E, n, n, n))
    u = g.uniform(-1, 1, (E, n, n, n))
    want = env["oracle"].inv_helmholtz(S, D, u)
    got = env["ops"].ekl_tpo_inv_helmholtz(to_dev(env, S), to_dev(env, D), to_dev(env, u))
    err = env["oracle"].rel_err_per_element(got.cpu().numpy(), want)
    assert err.max() <= TOL64


@pytest.mark.parametrize("n,E", [(3, 65), (4, 65), (5, 1001), (8, 65), (12, 65), (13, 402),
                                 (14, 65), (14, 1500), (15, 33), (16, 300), (20, 9)])
def test_inv_helmholtz_f32(env, n, E):
    torch = env["torch"]
    S, D, u = synth_ih(n, E, 77 + n)
    S32, D32, u32 = (x.astype(np.float32) for x in (S, D, u))
    want = env["oracle"].inv_helmholtz(S32, D32, u32)          # widened, computed in fp64
    got = env["ops"].ekl_tpo_inv_helmholtz_f32(to_dev(env, S32), to_dev(env, D32), to_dev(env, u32))
    assert got.dtype == torch.float32
    err = env["oracle"].rel_err_per_element(got.cpu().numpy().astype(np.float64), want)
    assert err.max() <= TOL32


@pytest.mark.parametrize("n", [8, 10, 12, 14, 16])
@pytest.mark.parametrize("E", [1, 2, 777, 20001])
def test_inv_helmholtz_f32_split_tf32_path(env, n, E):
    """Even extents 8..16 in single precision run on the TF32 tensor path with split operands
    (three tensor steps per product).  A dropped or wrong cross term would leave an error of
    1e-4 or more, so the 1e-5 bar is the check; E spans one element, one batch, an odd count
    and many batches per CTA.  A non-orthogonal, non-symmetric S separates S from its
    transpose in both halves."""
    g = rng(900 + n)
    S = (g.standard_normal((n, n)) / np.sqrt(n)).astype(np.float32)
    D = g.uniform(0.13, 1.25, (E, n, n, n)).astype(np.float32)
    u = g.uniform(-1, 1, (E, n, n, n)).astype(np.float32)
    dS, dD, du = to_dev(env, S), to_dev(env, D), to_dev(env, u)
    got = env["ops"].ekl_tpo_inv_helmholtz_f32(dS, dD, du)
    sample = np.unique(np.concatenate([np.arange(min(E, 300)), np.arange(max(E - 300, 0), E)]))
    want = env["oracle"].inv_helmholtz(S, D[sample], u[sample])
    err = env["oracle"].rel_err_per_element(got.cpu().numpy()[sample].astype(np.float64), want)
    assert err.max() <= TOL32, (n, E, err.max())
    # in place, and the same bits on a second call
    again = env["ops"].ekl_tpo_inv_helmholtz_f32(dS, dD, du, out=du)
    assert again.data_ptr() == du.data_ptr()
    assert env["torch"].equal(again, got)


def test_inv_helmholtz_f32_unaligned_u_leaves_the_tf32_path(env):
    """The TF32 path bulk-copies u and needs it 16-byte aligned; a view that starts 4 bytes
    into an allocation takes another kernel and must give the same answer to tolerance."""
    torch = env["torch"]
    n, E = 14, 37
    g = rng(4242)
    S = (g.standard_normal((n, n)) / np.sqrt(n)).astype(np.float32)
    D = g.uniform(0.13, 1.25, (E, n, n, n)).astype(np.float32)
    u = g.uniform(-1, 1, (E, n, n, n)).astype(np.float32)
    flat = torch.empty(E * n ** 3 + 1, dtype=torch.float32, device=env["dev"])
    du = flat[1:].view(E, n, n, n)
    du.copy_(torch.from_numpy(u))
    assert du.data_ptr() % 16 == 4
    got = env["ops"].ekl_tpo_inv_helmholtz_f32(to_dev(env, S), to_dev(env, D), du)
    want = env["oracle"].inv_helmholtz(S, D, u)
    err = env["oracle"].rel_err_per_element(got.cpu().numpy().astype(np.float64), want)
    assert err.max() <= TOL32


@pytest.mark.parametrize("n", [4, 8, 12, 14])
def test_inv_helmholtz_exact_special_cases(env, n):
    """S = I gives D∘u bit for bit (every extra term is ×0, +0); a permutation matrix
    gives an exact permuted, scaled copy."""
    g = rng(5 + n)
    E = 19
    D = g.uniform(0.1, 1.3, (E, n, n, n))
    u = g.uniform(-1, 1, (E, n, n, n))
    got = env["ops"].ekl_tpo_inv_helmholtz(to_dev(env, np.eye(n)), to_dev(env, D), to_dev(env, u))
    assert np.array_equal(got.cpu().numpy(), D * u)
    perm = g.permutation(n)
    S = np.zeros((n, n))
    S[np.arange(n), perm] = 1.0
    want = env["oracle"].inv_helmholtz(S, D, u)
    got = env["ops"].ekl_tpo_inv_helmholtz(to_dev(env, S), to_dev(env, D), to_dev(env, u))
    assert np.array_equal(got.cpu().numpy(), want)


@pytest.mark.parametrize("n,E", [(4, 64), (8, 777), (12, 150), (14, 149), (14, 300)])
def test_inv_helmholtz_in_place_guards_and_repeatability(env, n, E):
    """v == u in place; canaries around v untouched; NaN-prefilled output fully
    overwritten; two runs bitwise identical (no races, no unwritten outputs)."""
    torch = env["torch"]
    S, D, u = synth_ih(n, E, 9 + n)
    want = env["oracle"].inv_helmholtz(S, D, u)
    Sd, Dd, ud = to_dev(env, S), to_dev(env, D), to_dev(env, u)
    pad = 512
    big = torch.full((E * n ** 3 + 2 * pad,), float("nan"), dtype=torch.float64, device=env["dev"])
    big[:pad] = 12345.0
    big[-pad:] = 54321.0
    out = big[pad:-pad].view(E, n, n, n)
    env["ops"].ekl_tpo_inv_helmholtz(Sd, Dd, ud, out=out)
    first = out.clone()
    out.fill_(float("nan"))
    env["ops"].ekl_tpo_inv_helmholtz(Sd, Dd, ud, out=out)
    assert torch.equal(first, out)
    assert bool((big[:pad] == 12345.0).all()) and bool((big[-pad:] == 54321.0).all())
    assert env["oracle"].rel_err_per_element(out.cpu().numpy(), want).max() <= TOL64
    inplace = ud.clone()
    env["ops"].ekl_tpo_inv_helmholtz(Sd, Dd, inplace, out=inplace)
    assert torch.equal(inplace, first)


def test_element_permutation_and_batch_independence(env):
    torch = env["torch"]
    n, E = 14, 130
    S, D, u = synth_ih(n, E, 4242)
    Sd, Dd, ud = to_dev(env, S), to_dev(env, D), to_dev(env, u)
    full = env["ops"].ekl_tpo_inv_helmholtz(Sd, Dd, ud)
    p = torch.from_numpy(rng(1).permutation(E)).to(env["dev"])
    shuf = env["ops"].ekl_tpo_inv_helmholtz(Sd, Dd[p].contiguous(), ud[p].contiguous())
    assert torch.equal(shuf, full[p])


@pytest.mark.parametrize("n", [8, 12, 14])
def test_inv_helmholtz_unaligned_u_takes_the_general_kernel(env, n):
    """u offset by one double is only 8-byte aligned: the tensor path (which bulk-copies u)
    is skipped and the general kernel must give the same answer."""
    torch = env["torch"]
    E = 21
    S, D, u = synth_ih(n, E, 31 + n)
    want = env["oracle"].inv_helmholtz(S, D, u)
    Sd, Dd = to_dev(env, S), to_dev(env, D)
    store = torch.zeros(E * n ** 3 + 1, dtype=torch.float64, device=env["dev"])
    ud = store[1:].view(E, n, n, n)
    ud.copy_(to_dev(env, u))
    assert ud.data_ptr() % 16 == 8
    got = env["ops"].ekl_tpo_inv_helmholtz(Sd, Dd, ud)
    assert env["oracle"].rel_err_per_element(got.cpu().numpy(), want).max() <= TOL64
    aligned = env["ops"].ekl_tpo_inv_helmholtz(Sd, Dd, ud.clone())
    assert env["oracle"].rel_err_per_element(aligned.cpu().numpy(), want).max() <= TOL64


@pytest.mark.parametrize("n,E", [(5, 4099), (9, 2500), (13, 1201), (15, 999), (16, 700), (11, 1)])
def test_inv_helmholtz_many_batches_per_cta(env, n, E):
    """Enough elements that every persistent CTA loops over several batches and the last
    batch is partly filled; u and D deliberately only 8-byte aligned for odd n."""
    torch = env["torch"]
    S, D, u = synth_ih(n, E, 7000 + n)
    want = env["oracle"].inv_helmholtz(S, D, u)
    off = 1 if n % 2 else 0
    ubuf = torch.zeros(E * n ** 3 + 1, dtype=torch.float64, device=env["dev"])
    dbuf = torch.zeros(E * n ** 3 + 1, dtype=torch.float64, device=env["dev"])
    ud = ubuf[off:off + E * n ** 3].view(E, n, n, n)
    dd = dbuf[off:off + E * n ** 3].view(E, n, n, n)
    ud.copy_(to_dev(env, u))
    dd.copy_(to_dev(env, D))
    got = env["ops"].ekl_tpo_inv_helmholtz(to_dev(env, S), dd, ud)
    torch.cuda.synchronize()
    err = env["oracle"].rel_err_per_element(got.cpu().numpy(), want)
    assert err.max() <= TOL64, (n, E, err.max())


@pytest.mark.parametrize("n,E", [(14, 3001), (12, 2000), (9, 1500), (8, 5000)])
def test_inv_helmholtz_in_place_with_many_batches_per_cta(env, n, E):
    """v == u while every persistent CTA streams several batches: a batch's u must be on chip
    before its v is written, and no CTA may touch another one's elements."""
    torch = env["torch"]
    S, D, u = synth_ih(n, E, 9100 + n)
    Sd, Dd, ud = to_dev(env, S), to_dev(env, D), to_dev(env, u)
    ref = env["ops"].ekl_tpo_inv_helmholtz(Sd, Dd, ud)
    inplace = ud.clone()
    env["ops"].ekl_tpo_inv_helmholtz(Sd, Dd, inplace, out=inplace)
    torch.cuda.synchronize()
    assert torch.equal(inplace, ref)
    sample = slice(E - 40, E)
    want = env["oracle"].inv_helmholtz(S, D[sample], u[sample])
    assert env["oracle"].rel_err_per_element(ref[sample].cpu().numpy(), want).max() <= TOL64


def test_no_device_error_flags_after_all_this(env):
    lib = env["ops"].library()
    lib.ekl_tpo_device_error_flags.restype = __import__("ctypes").c_int
    assert lib.ekl_tpo_device_error_flags() == 0


# --------------------------------------------------------------------------- forward operator

SHAPES = [((2, 3, 4), (5, 2, 3)), ((8, 8, 8), (12, 12, 12)), ((12, 12, 12), (8, 8, 8)),
          ((1, 1, 1), (1, 1, 1)), ((7, 1, 5), (2, 9, 3)), ((4, 4, 4), (4, 4, 4)),
          ((14, 14, 14), (14, 14, 14)), ((5, 6, 7), (7, 6, 5)), ((16, 3, 9), (3, 16, 2))]


@pytest.mark.parametrize("nn,mm", SHAPES)
@pytest.mark.parametrize("E", [1, 3, 130])
def test_apply_f64(env, nn, mm, E):
    g = rng(hash((nn, mm, E)) % 10000)
    A, B, C = (g.standard_normal((mm[d], nn[d])) / np.sqrt(nn[d]) for d in range(3))
    u = g.uniform(-1, 1, (E,) + nn)
    want = env["oracle"].tpo_apply(A, B, C, u)
    got = env["ops"].ekl_tpo_apply(*(to_dev(env, x) for x in (A, B, C, u)))
    assert tuple(got.shape) == (E,) + mm
    assert env["oracle"].rel_err_per_element(got.cpu().numpy(), want).max() <= TOL64


@pytest.mark.parametrize("n,m", [(4, 6), (6, 4), (10, 14), (14, 16), (16, 16), (16, 4), (12, 12),
                                 (8, 8), (14, 10), (6, 16)])
@pytest.mark.parametrize("E", [1, 2, 3, 257])
def test_apply_f64_cubic_pairs_on_the_tensor_path(env, n, m, E):
    g = rng(100 * n + m + E)
    A, B, C = (g.standard_normal((m, n)) / np.sqrt(n) for _ in range(3))
    u = g.uniform(-1, 1, (E, n, n, n))
    want = env["oracle"].tpo_apply(A, B, C, u)
    got = env["ops"].ekl_tpo_apply(*(to_dev(env, x) for x in (A, B, C, u)))
    env["torch"].cuda.synchronize()
    assert env["oracle"].rel_err_per_element(got.cpu().numpy(), want).max() <= TOL64


ANISO = [((8, 8, 8), (12, 12, 8)), ((8, 8, 8), (8, 8, 12)), ((12, 12, 12), (8, 8, 12)),
         ((12, 12, 8), (8, 8, 12)), ((8, 10, 12), (12, 10, 8)), ((8, 10, 12), (8, 10, 12)),
         ((6, 8, 10), (10, 8, 6)), ((14, 12, 8), (8, 12, 14))]


@pytest.mark.parametrize("nn,mm", ANISO)
@pytest.mark.parametrize("E", [1, 2, 3, 257, 4001])
def test_apply_f64_non_cubic_shapes_on_the_tensor_path(env, nn, mm, E):
    """Three different operators on all-distinct extents: any axis mix-up fails.  E = 4001 gives
    every CTA several batches (the dynamic deal of batches)."""
    g = rng(hash((nn, mm)) % 9973 + E)
    A, B, C = (g.standard_normal((mm[d], nn[d])) / np.sqrt(nn[d]) for d in range(3))
    u = g.uniform(-1, 1, (E,) + nn)
    want = env["oracle"].tpo_apply(A, B, C, u)
    v = env["torch"].full((E,) + mm, float("nan"), dtype=env["torch"].float64, device=env["dev"])
    got = env["ops"].ekl_tpo_apply(*(to_dev(env, x) for x in (A, B, C, u)), out=v)
    env["torch"].cuda.synchronize()
    assert env["oracle"].rel_err_per_element(got.cpu().numpy(), want).max() <= TOL64
    # the same shape through the general kernel (an unaligned u falls back to it) agrees
    if E == 257:
        buf = env["torch"].zeros(u.size + 1, dtype=env["torch"].float64, device=env["dev"])
        uu = buf[1:].view(u.shape)
        uu.copy_(to_dev(env, u))
        got2 = env["ops"].ekl_tpo_apply(*(to_dev(env, x) for x in (A, B, C)), uu)
        assert env["oracle"].rel_err_per_element(got2.cpu().numpy(), want).max() <= TOL64


@pytest.mark.parametrize("nn,mm", ANISO)
def test_apply_f32_non_cubic_shapes(env, nn, mm):
    """The non-cubic tensor-path shapes with fp32 fields (widened on chip, fp64 arithmetic)."""
    g = rng(hash((mm, nn)) % 9973)
    E = 203
    A, B, C = ((g.standard_normal((mm[d], nn[d])) / np.sqrt(nn[d])).astype(np.float32)
               for d in range(3))
    u = g.uniform(-1, 1, (E,) + nn).astype(np.float32)
    want = env["oracle"].tpo_apply(A, B, C, u)
    got = env["ops"].ekl_tpo_apply_f32(*(to_dev(env, x) for x in (A, B, C, u)))
    err = env["oracle"].rel_err_per_element(got.cpu().numpy().astype(np.float64), want)
    assert err.max() <= TOL32


ODD_CUBIC = [(5, 5), (7, 7), (9, 9), (11, 11), (13, 13), (15, 15), (5, 7), (7, 5), (7, 9), (9, 7),
             (9, 11), (11, 9), (11, 13), (13, 11), (13, 15), (15, 13), (5, 8), (8, 5), (6, 9), (9, 6),
             (7, 11), (11, 7), (9, 14), (14, 9), (10, 15), (15, 10), (4, 5), (5, 4), (5, 6), (6, 5),
             (6, 7), (7, 6), (7, 8), (8, 7), (8, 9), (9, 8), (9, 10), (10, 9)]


@pytest.mark.parametrize("n,m", ODD_CUBIC)
def test_apply_cubic_shapes_with_an_odd_extent(env, n, m):
    """Cubic n -> m forward operators where n or m is odd (tensor-path instances whose fields
    have odd planes or odd rows): three different matrices, element counts that leave a partly
    filled batch and that give every CTA several batches, fp64 and fp32 fields, and u starting
    8 bytes off a 16-byte boundary (allowed when a plane of u is an odd number of values)."""
    torch = env["torch"]
    g = rng(100 * n + m)
    A, B, C = (g.standard_normal((m, n)) / np.sqrt(n) for _ in range(3))
    for E in (1, 3, 4001):
        u = g.uniform(-1, 1, (E, n, n, n))
        want = env["oracle"].tpo_apply(A, B, C, u)
        v = torch.full((E, m, m, m), float("nan"), dtype=torch.float64, device=env["dev"])
        got = env["ops"].ekl_tpo_apply(*(to_dev(env, x) for x in (A, B, C, u)), out=v)
        torch.cuda.synchronize()
        assert env["oracle"].rel_err_per_element(got.cpu().numpy(), want).max() <= TOL64, E
    E = 77
    u = g.uniform(-1, 1, (E, n, n, n))
    want = env["oracle"].tpo_apply(A, B, C, u)
    buf = torch.zeros(u.size + 1, dtype=torch.float64, device=env["dev"])
    uu = buf[1:].view(u.shape)
    uu.copy_(to_dev(env, u))
    got = env["ops"].ekl_tpo_apply(*(to_dev(env, x) for x in (A, B, C)), uu)
    assert env["oracle"].rel_err_per_element(got.cpu().numpy(), want).max() <= TOL64
    A32, B32, C32, u32 = (x.astype(np.float32) for x in (A, B, C, u))
    want32 = env["oracle"].tpo_apply(A32, B32, C32, u32)
    got32 = env["ops"].ekl_tpo_apply_f32(*(to_dev(env, x) for x in (A32, B32, C32, u32)))
    err = env["oracle"].rel_err_per_element(got32.cpu().numpy().astype(np.float64), want32)
    assert err.max() <= TOL32
    assert env["ops"].library().ekl_tpo_device_error_flags() == 0


@pytest.mark.parametrize("nn,mm", SHAPES[:3])
def test_apply_f32(env, nn, mm):
    g = rng(3)
    E = 50
    A, B, C = ((g.standard_normal((mm[d], nn[d])) / np.sqrt(nn[d])).astype(np.float32)
               for d in range(3))
    u = g.uniform(-1, 1, (E,) + nn).astype(np.float32)
    want = env["oracle"].tpo_apply(A, B, C, u)
    got = env["ops"].ekl_tpo_apply_f32(*(to_dev(env, x) for x in (A, B, C, u)))
    err = env["oracle"].rel_err_per_element(got.cpu().numpy().astype(np.float64), want)
    assert err.max() <= TOL32


@pytest.mark.parametrize("n", [8, 10, 12, 14, 16])
@pytest.mark.parametrize("m", [8, 10, 12, 14, 16])
def test_apply_f32_split_tf32_path(env, n, m):
    """Cubic n -> m forward operators with even extents 8..16 in single precision run on the
    TF32 tensor path with split operands; three different matrices separate the axes, an odd
    element count leaves a partly filled batch."""
    g = rng(3000 + 20 * n + m)
    E = 515
    A, B, C = ((g.standard_normal((m, n)) / np.sqrt(n)).astype(np.float32) for _ in range(3))
    u = g.uniform(-1, 1, (E, n, n, n)).astype(np.float32)
    got = env["ops"].ekl_tpo_apply_f32(*(to_dev(env, x) for x in (A, B, C, u)))
    want = env["oracle"].tpo_apply(A, B, C, u)
    err = env["oracle"].rel_err_per_element(got.cpu().numpy().astype(np.float64), want)
    assert err.max() <= TOL32, (n, m, err.max())


def test_apply_selection_matrices_gather_exactly(env):
    g = rng(8)
    nn, mm = (8, 8, 8), (12, 12, 12)
    rows = [g.integers(0, nn[d], size=mm[d]) for d in range(3)]
    A, B, C = (np.eye(nn[d])[rows[d]] for d in range(3))
    u = g.uniform(-1, 1, (40,) + nn)
    want = u[:, rows[0]][:, :, rows[1]][:, :, :, rows[2]]
    got = env["ops"].ekl_tpo_apply(*(to_dev(env, x) for x in (A, B, C, u)))
    assert np.array_equal(got.cpu().numpy(), want)


def test_apply_guards_and_repeatability(env):
    torch = env["torch"]
    g = rng(12)
    nn, mm, E = (8, 8, 8), (12, 12, 12), 333
    A, B, C = (g.standard_normal((mm[d], nn[d])) / np.sqrt(nn[d]) for d in range(3))
    u = g.uniform(-1, 1, (E,) + nn)
    dev = [to_dev(env, x) for x in (A, B, C, u)]
    pad = 512
    big = torch.full((E * 12 ** 3 + 2 * pad,), float("nan"), dtype=torch.float64, device=env["dev"])
    big[:pad] = 1.5
    big[-pad:] = 2.5
    out = big[pad:-pad].view(E, 12, 12, 12)
    env["ops"].ekl_tpo_apply(*dev, out=out)
    first = out.clone()
    out.fill_(float("nan"))
    env["ops"].ekl_tpo_apply(*dev, out=out)
    assert torch.equal(first, out)
    assert bool((big[:pad] == 1.5).all()) and bool((big[-pad:] == 2.5).all())
    assert not bool(torch.isnan(out).any())


# --------------------------------------------------------------------------- binding / status paths

def test_runtime_argument_errors_raise(env):
    torch, ops = env["torch"], env["ops"]
    n, E = 4, 8
    S = torch.eye(n, dtype=torch.float64, device=env["dev"])
    u = torch.zeros(E, n, n, n, dtype=torch.float64, device=env["dev"])
    with pytest.raises(ops.EklTpoError, match="OVERLAP"):
        ops.ekl_tpo_inv_helmholtz(S, u, u.clone(), out=u)        # D aliases v
    with pytest.raises(TypeError):
        ops.ekl_tpo_inv_helmholtz(S.float(), u, u)
    with pytest.raises(TypeError):
        ops.ekl_tpo_inv_helmholtz(S.cpu(), u, u)
    with pytest.raises(ValueError):
        ops.ekl_tpo_inv_helmholtz(S, u, u.transpose(1, 2))
    big = torch.zeros(1, 26, 26, 26, dtype=torch.float64, device=env["dev"])
    with pytest.raises(ops.EklTpoError, match="UNSUPPORTED"):
        ops.ekl_tpo_inv_helmholtz(torch.eye(26, dtype=torch.float64, device=env["dev"]), big, big)
    empty = torch.zeros(0, n, n, n, dtype=torch.float64, device=env["dev"])
    assert ops.ekl_tpo_inv_helmholtz(S, empty, empty).shape == (0, n, n, n)


def test_device_input_generators_match_the_host_bit_for_bit(env):
    inputs = env["inputs"]
    for idx in (0, 1, 4, 5):
        wl = inputs.CONFIGS[idx]
        e0, e1 = 5, min(wl.E, 45)
        host = inputs.host_case(wl, e0, e1)
        dev = inputs.device_case(wl, env["dev"], e0, e1)
        for key in host:
            h = host[key]
            d = dev[key].cpu().numpy() if hasattr(dev[key], "cpu") else dev[key]
            assert np.array_equal(h, d), (idx, key)


# --------------------------------------------------------------------------- element independence

@pytest.mark.parametrize("n,dtype", [(14, "f64"), (8, "f64"), (5, "f64"), (3, "f64"), (12, "f64"),
                                     (14, "f32"), (8, "f32"), (7, "f32")])
def test_elements_are_independent(env, n, dtype):
    """The elements of a batch share tensor tiles and shared-memory buffers, but every result
    depends on its own element only: with NaN and Inf written into a few elements of u and D,
    every other element of v is bit-identical to the clean run, and the poisoned ones are not
    finite.  Covers both neighbours in a batch of two, a whole batch, and the last (partly
    filled) batch."""
    torch = env["torch"]
    E = 1203
    S, D, u = synth_ih(n, E, 31 * n)
    tdt = torch.float64 if dtype == "f64" else torch.float32
    fn = env["ops"].ekl_tpo_inv_helmholtz if dtype == "f64" else env["ops"].ekl_tpo_inv_helmholtz_f32
    Sd, Dd, ud = (to_dev(env, x, tdt) for x in (S, D, u))
    clean = fn(Sd, Dd, ud).clone()
    bad_u = [0, 5, 400, 401, E - 1]
    bad_d = [77, 800]
    up, Dp = ud.clone(), Dd.clone()
    for k, e in enumerate(bad_u):
        up[e].view(-1)[(13 * k) % n ** 3] = float("nan") if k % 2 == 0 else float("inf")
    for e in bad_d:
        Dp[e].view(-1)[n ** 3 - 1] = float("nan")
    got = fn(Sd, Dp, up)
    torch.cuda.synchronize()
    bad = torch.zeros(E, dtype=torch.bool, device=env["dev"])
    bad[bad_u + bad_d] = True
    assert torch.equal(got[~bad], clean[~bad])
    assert not bool(torch.isfinite(got[bad]).all(dim=(1, 2, 3)).any())


def test_forward_and_convection_elements_are_independent(env):
    torch = env["torch"]
    g = rng(99)
    E = 777
    A, B, C = (g.standard_normal((12, 8)) / 3 for _ in range(3))
    u = g.uniform(-1, 1, (E, 8, 8, 8))
    dev = [to_dev(env, x) for x in (A, B, C, u)]
    clean = env["ops"].ekl_tpo_apply(*dev).clone()
    up = dev[3].clone()
    for e in (1, 300, E - 1):
        up[e, 3, 4, 5] = float("nan")
    got = env["ops"].ekl_tpo_apply(dev[0], dev[1], dev[2], up)
    bad = torch.zeros(E, dtype=torch.bool, device=env["dev"])
    bad[[1, 300, E - 1]] = True
    assert torch.equal(got[~bad], clean[~bad])
    assert bool(torch.isnan(got[bad]).any(dim=(1, 2, 3)).all())
    # convection: a NaN in M[e] reaches all three components of element e and nothing else
    nq, nv, Ec = 12, 8, 333
    Dvq, Ivq = (to_dev(env, g.standard_normal((nv, nq)) / 3) for _ in range(2))
    M = to_dev(env, g.uniform(0.5, 1.5, (Ec, nq, nq, nq)))
    P = to_dev(env, g.uniform(-1, 1, (3, 3, Ec, nq, nq, nq)))
    clean = env["ops"].ekl_tpo_convection(Dvq, Ivq, M, P).clone()
    Mp = M.clone()
    Mp[100, 0, 0, 0] = float("nan")
    Pp = P.clone()
    Pp[1, 2, 200, 5, 5, 5] = float("inf")
    got = env["ops"].ekl_tpo_convection(Dvq, Ivq, Mp, Pp)
    torch.cuda.synchronize()
    same = torch.ones(3, Ec, dtype=torch.bool, device=env["dev"])
    same[:, 100] = False
    same[1, 200] = False
    assert torch.equal(got[same], clean[same])
    assert not bool(torch.isfinite(got[~same]).all(dim=(1, 2, 3)).any())


@pytest.mark.parametrize("n,dtype,k", [(14, "f64", 400), (14, "f64", -400), (9, "f64", 300),
                                       (3, "f64", -300), (14, "f32", 40), (12, "f32", -40),
                                       (7, "f32", 30)])
def test_scaling_by_a_power_of_two_is_exact(env, n, dtype, k):
    """The operator is linear in u and in D, and a power of two changes no rounding while
    nothing overflows or underflows: v(2^k u, D) = v(u, 2^k D) = 2^k v(u, D) bit for bit.
    A hidden conversion to a narrower format (or a fused multiply that is not there in the
    other run) would break it; so would the split of fp32 values into TF32 parts if it were
    not scale invariant."""
    torch = env["torch"]
    E = 129
    S, D, u = synth_ih(n, E, 17 * n + 3)
    tdt = torch.float64 if dtype == "f64" else torch.float32
    fn = env["ops"].ekl_tpo_inv_helmholtz if dtype == "f64" else env["ops"].ekl_tpo_inv_helmholtz_f32
    Sd, Dd, ud = (to_dev(env, x, tdt) for x in (S, D, u))
    base = fn(Sd, Dd, ud)
    f = 2.0 ** k
    assert torch.equal(fn(Sd, Dd, ud * f), base * f)
    assert torch.equal(fn(Sd, Dd * f, ud), base * f)


@pytest.mark.parametrize("n,E", [(5, 4099), (7, 3001), (9, 2501), (11, 1801), (13, 1201), (5, 6), (9, 4)])
def test_inv_helmholtz_odd_n_aligned_fields_many_batches(env, n, E):
    """Odd n with 16-byte aligned fields (the other odd-n cases offset them by 8 bytes), an odd E
    that leaves a partly filled last batch, several batches per CTA; also in place."""
    torch = env["torch"]
    S, D, u = synth_ih(n, E, 9100 + n)
    want = env["oracle"].inv_helmholtz(S, D, u)
    Sd, Dd, ud = to_dev(env, S), to_dev(env, D), to_dev(env, u)
    assert ud.data_ptr() % 16 == 0
    got = env["ops"].ekl_tpo_inv_helmholtz(Sd, Dd, ud)
    env["torch"].cuda.synchronize()
    assert env["oracle"].rel_err_per_element(got.cpu().numpy(), want).max() <= TOL64
    inplace = ud.clone()
    env["ops"].ekl_tpo_inv_helmholtz(Sd, Dd, inplace, out=inplace)
    assert torch.equal(inplace, got)
    assert env["ops"].library().ekl_tpo_device_error_flags() == 0
