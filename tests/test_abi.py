"""The C-ABI library loads, exports every symbol the header declares, and rejects bad
arguments on the host (no kernel is launched, so this runs without a GPU)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2007_12792_b200 import build, binding
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dn_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    from paper_2007_12792_b200 import binding
    names = declared_symbols()
    assert len(names) >= 9
    for n in names:
        assert hasattr(L, n), n
    assert set(binding.EXPORTS) == set(names)


def test_status_strings(L):
    from paper_2007_12792_b200 import binding
    seen = {binding.status_string(s) for s in range(0, 8)}
    assert len(seen) == 8 and binding.status_string(0) == "ok"


def test_host_side_validation(L):
    from paper_2007_12792_b200 import binding as B
    fake = 0x1000  # never dereferenced: validation fails first

    def prob(**kw):
        p = B.DnProblem()
        p.grid = B.DnGrid(kw.get("dim", 2), kw.get("nx", 8), kw.get("ny", 8), kw.get("nz", 1))
        p.batch = kw.get("batch", 1)
        p.nu_mode = kw.get("nu_mode", B.DN_NU_KL_GAUSS)
        p.kl_modes = kw.get("kl_modes", 2)
        p.kl_w = kw.get("kl_w", fake)
        p.nu = kw.get("nu", None)
        return p

    def eg(p, u=fake, r=fake * 1024, ws=fake * 4096, ws_bytes=1 << 30):
        return L.dn_energy_grad(C.byref(p), u, None, None, r, ws, ws_bytes, None)

    assert L.dn_workspace_bytes(C.byref(prob())) > 0
    assert L.dn_workspace_bytes(C.byref(prob())) % 256 == 0
    assert L.dn_host_staging_bytes(C.byref(prob())) > L.dn_workspace_bytes(C.byref(prob()))
    assert L.dn_workspace_bytes(None) == 0
    assert L.dn_energy_grad(None, fake, None, None, fake, fake, 0, None) == B.DN_ERR_NULL
    assert eg(prob(dim=4)) == B.DN_ERR_DIM
    assert eg(prob(nx=1)) == B.DN_ERR_SIZE
    assert eg(prob(dim=3, nz=1)) == B.DN_ERR_SIZE
    assert eg(prob(batch=0)) == B.DN_ERR_SIZE
    assert eg(prob(nx=40000)) == B.DN_ERR_SIZE
    assert eg(prob(nu_mode=7)) == B.DN_ERR_MODE
    assert eg(prob(kl_modes=0)) == B.DN_ERR_MODE
    assert eg(prob(kl_modes=B.DN_MAX_KL_MODES + 1)) == B.DN_ERR_MODE
    assert eg(prob(kl_w=None)) == B.DN_ERR_NULL
    assert eg(prob(nu_mode=B.DN_NU_NODAL, nu=None)) == B.DN_ERR_NULL
    assert eg(prob(), u=None) == B.DN_ERR_NULL
    assert eg(prob(), r=None) == B.DN_ERR_NULL
    assert eg(prob(), r=fake + 16) == B.DN_ERR_ALIAS
    assert eg(prob(), ws=None) == B.DN_ERR_WORKSPACE
    assert eg(prob(), ws=fake * 4096 + 8) == B.DN_ERR_WORKSPACE
    assert eg(prob(), ws_bytes=16) == B.DN_ERR_WORKSPACE
    assert L.dn_energy(C.byref(prob()), fake, None, fake * 4096, 1 << 30, None) == B.DN_ERR_NULL
    g = B.DnGrid(2, 8, 8, 1)
    assert L.dn_kl_field(C.byref(g), 1, 0, fake, fake, None) == B.DN_ERR_MODE
    assert L.dn_kl_field(C.byref(g), 1, 2, None, fake, None) == B.DN_ERR_NULL
    assert L.dn_kl_field(C.byref(B.DnGrid(5, 8, 8, 1)), 1, 2, fake, fake, None) == B.DN_ERR_DIM
    assert L.dn_apply_bc(C.byref(g), 1, 1.0, 0.0, 3, fake, None) == B.DN_ERR_MODE
    assert L.dn_apply_bc(C.byref(g), 0, 1.0, 0.0, 0, fake, None) == B.DN_ERR_SIZE
    assert L.dn_apply_bc(C.byref(g), 1, 1.0, 0.0, 0, None, None) == B.DN_ERR_NULL
    assert L.dn_energy_grad_host(C.byref(prob()), fake, None, None, fake, None, 0, None) == B.DN_ERR_WORKSPACE
    assert L.dn_launches_per_call(C.byref(prob())) == 3
    assert L.dn_launches_per_call(C.byref(prob(dim=9))) == 0
    assert L.dn_path_name(C.byref(prob(nx=7))) == b"generic"


def test_entry_point_without_workspace_refuses_on_the_host(L):
    """dn_energy_grad_static decides on the host, before touching the device, whether its built-in 1 MiB of scratch
    is enough: wide 2D grids whose strip-kernel table does not fit and that no other kernel family can serve
    within the limit are refused with DN_ERR_WORKSPACE (they used to divide by zero in the tiled geometry)."""
    from paper_2007_12792_b200 import binding as B
    fake = 0x100000

    def prob(nx, ny, batch, m, mode=B.DN_NU_KL_GAUSS, dim=2, nz=1):
        p = B.DnProblem()
        p.grid = B.DnGrid(dim, nx, ny, nz)
        p.batch = batch; p.nu_mode = mode; p.kl_modes = m; p.kl_w = fake
        p.nu = fake if mode == B.DN_NU_NODAL else None
        return p

    def st(p, u=fake, r=fake << 12):
        return L.dn_energy_grad_static(C.byref(p), u, None, None, r, None)

    assert st(prob(4096, 4096, 16, 6)) == B.DN_ERR_WORKSPACE
    assert st(prob(4096, 4096, 2, 6)) == B.DN_ERR_WORKSPACE
    assert st(prob(4096, 4096, 2, 6, mode=B.DN_NU_KL_NODAL)) == B.DN_ERR_WORKSPACE
    assert st(prob(8192, 64, 1, 8)) in (B.DN_ERR_WORKSPACE, B.DN_ERR_CUDA)   # fits or not (no device here), no crash
    assert st(prob(256, 256, 4, 3, dim=3, nz=256)) == B.DN_ERR_WORKSPACE   # 3D tile seams beyond 1 MiB
    assert st(prob(4001, 4001, 16, 2)) == B.DN_ERR_WORKSPACE               # any-size kernel: too many partials
    # validation comes first here too
    assert st(prob(4096, 4096, 16, 0)) == B.DN_ERR_MODE
    assert st(prob(64, 64, 2, 2), u=None) == B.DN_ERR_NULL
    assert st(prob(64, 64, 2, 2), r=fake + 64) == B.DN_ERR_ALIAS
    assert L.dn_energy_grad_static(C.byref(prob(64, 64, 2, 2)), fake, None, None, None, None) == B.DN_ERR_NULL


def test_kernel_family_and_launch_count_by_shape(L):
    """Which kernel family the fused call takes is decided on the host from the shape alone (pointer alignment aside)."""
    from paper_2007_12792_b200 import binding as B
    fake = 0x100000

    def prob(dim, nx, ny, nz, mode=B.DN_NU_KL_GAUSS, f=None, flags=0, batch=4, m=3):
        p = B.DnProblem()
        p.grid = B.DnGrid(dim, nx, ny, nz)
        p.batch = batch; p.nu_mode = mode; p.kl_modes = m; p.kl_w = fake
        p.nu = fake if mode == B.DN_NU_NODAL else None
        p.f = f; p.flags = flags
        return p

    name = lambda p: L.dn_path_name(C.byref(p)).decode()
    assert name(prob(2, 2048, 2048, 1)) == "strip2d" and name(prob(2, 256, 256, 1)) == "row2d"
    assert name(prob(2, 256, 256, 1, f=fake)) == "strip2d"              # nodal forcing: the strip kernel at every width
    assert name(prob(2, 260, 64, 1)) == "tiled2d" and name(prob(2, 132, 64, 1)) == "tiled2d"   # rows the row kernel's lanes do not tile
    for mode in (B.DN_NU_KL_GAUSS, B.DN_NU_NODAL, B.DN_NU_KL_NODAL):
        assert name(prob(2, 8, 2, 1, mode)) == "row2d" and name(prob(2, 128, 4000, 1, mode)) == "row2d"
    assert name(prob(2, 256, 256, 1, B.DN_NU_KL_NODAL)) == "row2d" and name(prob(2, 256, 256, 1, B.DN_NU_NODAL)) == "tiled2d"
    assert name(prob(2, 128, 64, 1, f=fake)) == "strip2d" and name(prob(2, 128, 8, 1, f=fake)) == "generic"   # ... on grids of 16 rows or more
    assert name(prob(2, 1030, 64, 1)) == "generic"
    for mode in (B.DN_NU_KL_GAUSS, B.DN_NU_NODAL, B.DN_NU_KL_NODAL):
        assert name(prob(3, 256, 256, 256, mode)) == "strip3d" and name(prob(3, 64, 64, 64, mode, f=fake)) == "strip3d"
        assert name(prob(3, 8, 2, 2, mode)) == "strip3d" and name(prob(3, 136, 9, 9, mode)) == "strip3d"
    assert name(prob(3, 260, 16, 16)) == "tiled3d" and name(prob(3, 260, 16, 16, B.DN_NU_KL_NODAL)) == "generic"
    assert name(prob(3, 512, 16, 16, B.DN_NU_NODAL)) == "tiled3d" and name(prob(3, 516, 16, 16)) == "generic"
    assert name(prob(3, 64, 64, 64, flags=B.DN_FORCE_GENERIC)) == "generic"
    # launches per call: tables, line polynomials, fused kernel, seam fix-up, finaliser
    assert L.dn_launches_per_call(C.byref(prob(3, 256, 256, 256))) == 5
    assert L.dn_launches_per_call(C.byref(prob(3, 256, 256, 256, B.DN_NU_NODAL))) == 3
    assert L.dn_launches_per_call(C.byref(prob(2, 2048, 2048, 1))) == 3
    # the scratch of a 3D problem: seams and the coefficient table, well below one field per sample
    p = prob(3, 256, 256, 256)
    assert 0 < L.dn_workspace_bytes(C.byref(p)) < 4 * 256 ** 3 * 4
    assert L.dn_cg_workspace_bytes(C.byref(p)) > 4 * 4 * 256 ** 3 * 4


def test_binding_rejects_host_tensors_and_missing_library(monkeypatch):
    import torch
    from paper_2007_12792_b200 import binding as B
    p = B.Problem(dim=2, nx=8, ny=8, batch=1, kl_modes=2, kl_w=torch.zeros(1, 2, 2))
    with pytest.raises(ValueError):
        p.c_struct()                      # host tensor where a device tensor is required: no CPU path
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/libdn.so")
    with pytest.raises(RuntimeError):
        B.lib()


def test_remembered_launch_geometry_does_not_leak_between_shapes(L):
    """Each kernel family keeps the launch geometry of the last shape it saw; alternating shapes, modes and forcing kinds
    must give what a first call gives (sizes differ between them, so a stale geometry would show)."""
    from paper_2007_12792_b200 import binding as B
    import threading
    fake = 0x100000

    def prob(dim, nx, ny, nz, batch, m, mode=B.DN_NU_KL_GAUSS, f=None):
        p = B.DnProblem()
        p.grid = B.DnGrid(dim, nx, ny, nz)
        p.batch = batch; p.nu_mode = mode; p.kl_modes = m; p.kl_w = fake
        p.nu = fake if mode == B.DN_NU_NODAL else None
        p.f = f
        return p

    probs = [prob(3, 256, 256, 256, 4, 3), prob(3, 64, 64, 64, 32, 2), prob(3, 256, 256, 256, 4, 3, B.DN_NU_NODAL),
             prob(3, 256, 256, 256, 4, 3, f=fake), prob(3, 256, 256, 256, 5, 3), prob(2, 2048, 2048, 1, 16, 6),
             prob(2, 2048, 2044, 1, 16, 6), prob(2, 256, 256, 1, 64, 4), prob(2, 256, 250, 1, 64, 4), prob(2, 64, 64, 1, 8, 2)]
    sizes = lambda: [(L.dn_workspace_bytes(C.byref(p)), L.dn_cg_workspace_bytes(C.byref(p)), L.dn_launches_per_call(C.byref(p)))
                     for p in probs]
    first = sizes()
    assert len(set(s[0] for s in first)) == len(first)          # every shape has its own scratch size
    assert sizes() == first and list(reversed([
        (L.dn_workspace_bytes(C.byref(p)), L.dn_cg_workspace_bytes(C.byref(p)), L.dn_launches_per_call(C.byref(p)))
        for p in reversed(probs)])) == first
    out = {}
    ts = [threading.Thread(target=lambda i=i: out.__setitem__(i, sizes())) for i in range(4)]   # per-thread memory
    [t.start() for t in ts]; [t.join() for t in ts]
    assert all(out[i] == first for i in range(4))
