"""GPU parity of the Burgers finite-difference loss (dn_burgers_loss_grad) against oracle/burgers.py."""
import numpy as np
import pytest
import torch

from oracle import burgers as ob
from paper_2007_12792_b200 import binding as B
from paper_2007_12792_b200 import inputs

pytestmark = pytest.mark.gpu

L_RTOL = 1e-5      # per sample |L - L*| <= L_RTOL |L*|  (same for L_p and L_b)
G_RTOL = 1e-5      # max |g - g*| <= G_RTOL max |g*|
T32 = float(np.float32(0.2))


def dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def run(inp, lam=1.0, gL=None, flags=0, want=("L", "parts", "g"), offset=0):
    p = B.Burgers(nx=inp.nx, nt=inp.nt, batch=inp.batch, c=dev(inp.c), T=T32, lam=lam, flags=flags)
    n = inp.u.size
    ubuf = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
    gbuf = torch.full((n + 8,), float("nan"), dtype=torch.float32, device="cuda")
    u = ubuf[offset:offset + n].view(p.shape)
    u.copy_(torch.from_numpy(inp.u))
    g = gbuf[offset:offset + n].view(p.shape) if "g" in want else None
    L = torch.full((inp.batch,), float("nan"), device="cuda") if "L" in want else None
    parts = torch.full((inp.batch, 2), float("nan"), device="cuda") if "parts" in want else None
    ws = B.new_burgers_workspace(p)
    B.dn_burgers_loss_grad(p, u, dev(gL), L, parts, g, ws)
    torch.cuda.synchronize()
    path = B.dn_burgers_path_name(p, u, g)
    f = lambda t: None if t is None else t.cpu().numpy().astype(np.float64)
    return f(L), f(parts), f(g), path


def check(inp, L, parts, g, lam=1.0, gL=None, samples=None):
    sel = slice(None) if samples is None else samples
    Lo, Lpo, Lbo, go = ob.loss_grad(inp.u[sel], inp.c[sel].astype(np.float64), T=T32, lam=lam,
                                    gL=None if gL is None else np.asarray(gL)[sel])
    if L is not None:
        assert np.all(np.abs(L[sel] - Lo) <= L_RTOL * np.abs(Lo)), (L[sel], Lo)
    if parts is not None:
        assert np.all(np.abs(parts[sel][:, 0] - Lpo) <= L_RTOL * np.abs(Lpo)), (parts[sel][:, 0], Lpo)
        assert np.all(np.abs(parts[sel][:, 1] - Lbo) <= L_RTOL * np.abs(Lbo)), (parts[sel][:, 1], Lbo)
    if g is not None:
        assert np.isfinite(g).all()
        err, scale = np.abs(g[sel] - go).max(), np.abs(go).max()
        assert err <= G_RTOL * scale, f"g max err {err:.3e} vs scale {scale:.3e} ({err / scale:.2e})"


# nx % 4 == 0 -> marching kernel; sizes span one warp, several warps with a ragged last warp, several chunks with a
# ragged last chunk, the smallest grid, and grids narrower than the warp's halo
MARCH_SIZES = [(4, 3, 2), (8, 5, 3), (120, 17, 2), (124, 40, 2), (256, 64, 3), (500, 300, 2), (1024, 70, 1), (12, 700, 2)]
GENERIC_SIZES = [(3, 3, 2), (5, 4, 1), (127, 33, 2), (258, 19, 2), (1001, 9, 1)]


@pytest.mark.parametrize("nx,nt,batch", MARCH_SIZES)
def test_march_kernel_matches_oracle(nx, nt, batch):
    inp = inputs.burgers_inputs(nx, nt, batch)
    L, parts, g, path = run(inp)
    assert path == "march"
    check(inp, L, parts, g)


@pytest.mark.parametrize("nx,nt,batch", GENERIC_SIZES + [(256, 64, 2)])
def test_any_size_kernel_matches_oracle(nx, nt, batch):
    inp = inputs.burgers_inputs(nx, nt, batch)
    L, parts, g, path = run(inp, flags=B.DN_FORCE_GENERIC)
    assert path == "generic"
    check(inp, L, parts, g)


def test_unaligned_pointers_take_the_any_size_kernel():
    inp = inputs.burgers_inputs(64, 32, 2)
    L, parts, g, path = run(inp, offset=1)
    assert path == "generic"
    check(inp, L, parts, g)


@pytest.mark.parametrize("flags", [0, B.DN_FORCE_GENERIC])
def test_options(flags):
    inp = inputs.burgers_inputs(248, 130, 3)
    gL = np.array([2.0, -0.5, 0.0], dtype=np.float32)
    L, parts, g, _ = run(inp, lam=0.3, gL=gL, flags=flags)
    check(inp, L, parts, g, lam=0.3, gL=gL)
    assert np.all(g[2] == 0.0)
    L2, _, g2, _ = run(inp, lam=0.3, flags=flags, want=("L",))          # loss only
    assert g2 is None and np.allclose(L2, L, rtol=1e-6, atol=0.0)
    _, parts3, g3, _ = run(inp, lam=0.0, flags=flags, want=("parts", "g"))
    check(inp, None, parts3, g3, lam=0.0)


def test_noise_free_and_large_noise_fields():
    for noise in (0.0, 0.3):
        inp = inputs.burgers_inputs(376, 90, 2, noise=noise)
        L, parts, g, _ = run(inp)
        check(inp, L, parts, g)


def test_deterministic_and_agrees_between_kernels():
    inp = inputs.burgers_inputs(512, 200, 2)
    a = run(inp)
    b = run(inp)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[2], b[2])
    c = run(inp, flags=B.DN_FORCE_GENERIC)
    assert np.abs(a[2] - c[2]).max() <= 2e-6 * np.abs(a[2]).max()


def test_validation():
    inp = inputs.burgers_inputs(16, 8, 1)
    p = B.Burgers(nx=16, nt=8, batch=1, c=dev(inp.c), T=T32)
    u = dev(inp.u)
    ws = B.new_burgers_workspace(p)
    with pytest.raises(B.DnError) as e:
        B.dn_burgers_loss_grad(p, u, None, None, None, u, ws)
    assert e.value.status == B.DN_ERR_ALIAS
    with pytest.raises(B.DnError) as e:
        B.dn_burgers_loss_grad(p, u, None, None, None, torch.empty_like(u), ws[:8])
    assert e.value.status == B.DN_ERR_WORKSPACE
    with pytest.raises(B.DnError) as e:
        B.dn_burgers_loss_grad(B.Burgers(nx=2, nt=8, batch=1, c=dev(inp.c)), u, None, None, None, torch.empty_like(u), ws)
    assert e.value.status == B.DN_ERR_SIZE
    assert B.dn_burgers_workspace_bytes(B.Burgers(nx=16, nt=8, batch=0, c=dev(inp.c))) == 0


def test_host_entry_point():
    inp = inputs.burgers_inputs(256, 96, 5)
    gL = np.array([1.0, 0.5, 2.0, -1.0, 0.25], dtype=np.float32)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).pin_memory()
    p = B.Burgers(nx=256, nt=96, batch=5, c=pin(inp.c), T=T32, lam=0.7)
    g_h = torch.full(p.shape, float("nan")).pin_memory()
    L_h = torch.full((5,), float("nan")).pin_memory()
    parts_h = torch.full((5, 2), float("nan")).pin_memory()
    staging = B.new_burgers_host_staging(p)
    B.dn_burgers_loss_grad_host(p, pin(inp.u), pin(gL), L_h, parts_h, g_h, staging)
    f = lambda t: t.numpy().astype(np.float64)
    check(inp, f(L_h), f(parts_h), f(g_h), lam=0.7, gL=gL)


def test_full_size_paper_example_on_sampled_samples():
    """1024 x 1024 outputs, minibatch 64 (the paper's first high-resolution example), in the launch configuration
    the benchmark times; the oracle scores three samples of the batch."""
    inp = inputs.burgers_inputs(1024, 1024, 64)
    L, parts, g, path = run(inp)
    assert path == "march"
    check(inp, L, parts, g, samples=[0, 31, 63])
    assert np.isfinite(L).all() and np.isfinite(g).all()
