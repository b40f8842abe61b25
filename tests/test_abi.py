"""The C-ABI library loads and exports every symbol the public header declares (no compute calls)."""
import ctypes
import os
import re

from paper_2602_14236_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(salicache_[a-z0-9_]+)\s*\(", src))
    return names


def test_library_exports_every_declared_symbol():
    lib = binding.lib()
    decl = _declared()
    assert {"salicache_flow_score", "salicache_saliency", "salicache_select", "salicache_pack_kv",
            "salicache_unpack_kv"} <= decl
    for name in sorted(decl):
        assert hasattr(lib, name), name
    assert set(binding.EXPORTS) <= decl


def test_params_struct_matches_the_header_defaults():
    p = binding.salicache_default_params()
    assert (p.H, p.W, p.patch, p.n_images) == (336, 336, 14, 1)
    assert (p.pyr_levels, p.poly_n, p.win, p.iters) == (3, 5, 15, 3)
    assert abs(p.poly_sigma - 1.2) < 1e-15 and abs(p.eps_det - 1e-3) < 1e-18
    assert (p.canny_lo, p.canny_hi, p.var_radius, p.hyst_max_iters) == (50, 150, 3, 4096)
    assert (p.L, p.heads, p.head_dim, p.group, p.patch_reuse) == (32, 32, 128, 128, 1)
    assert abs(p.tau_t - 0.5) < 1e-7 and abs(p.theta_R - 0.9) < 1e-7
    assert (round(p.tau_high, 4), round(p.tau_med, 4), round(p.tau_low, 4)) == (0.40, 0.36, 0.25)
    assert (p.color_norm, p.color_kappa, p.color_sigma_min) == (0, 1.0, 0.5)      # the struct's last fields: the layouts agree
    assert binding.lib().salicache_strerror(binding.E_CAPACITY).decode().startswith("tier pool")
    assert b"overwritten" in binding.lib().salicache_strerror(binding.E_EVICTED)


def test_host_side_argument_checks_need_no_device():
    lib = binding.lib()
    assert lib.salicache_default_params(None) == binding.E_NULL
    assert lib.salicache_create(None, None) == binding.E_NULL
    h = ctypes.c_void_p()
    bad = binding.salicache_default_params(win=7)
    assert lib.salicache_create(ctypes.byref(h), ctypes.byref(bad)) == binding.E_PARAM
    bad = binding.salicache_default_params(group=256)
    assert lib.salicache_create(ctypes.byref(h), ctypes.byref(bad)) == binding.E_PARAM
    bad = binding.salicache_default_params(H=300)
    assert lib.salicache_create(ctypes.byref(h), ctypes.byref(bad)) == binding.E_SHAPE
    assert lib.salicache_destroy(None) == binding.E_NULL
    assert lib.salicache_poll_status(None, None) == binding.E_NULL
