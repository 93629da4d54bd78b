"""Shows that the pins are not vacuous: each plausible mistake is planted into a COPY of the oracle's C
source (one text substitution), the copy is compiled, and at least one of the independent pins -- numpy
library routines, closed forms, torch.relu / torch.where -- must notice.  The shipped oracle is untouched."""
import ctypes
import os
import subprocess

import numpy as np
import pytest
import torch

from paper_2110_15362_b200 import workloads as W

SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle", "bt_oracle.c")

MUTANTS = {
    "msb_first_bit_order": ("(uint32_t)1 << (i & 31);                     /* push 1 bit */",
                            "(uint32_t)1 << (31 - (i & 31));"),
    "inclusive_prefix": ("if (i % CHUNK_ELEMS == 0) prefix[i / CHUNK_ELEMS] = j;\n        const unsigned char *e = src + i * (uint64_t)elem_size;\n        if (all_bytes_zero(e, elem_size)) {",
                         "if (i % CHUNK_ELEMS == CHUNK_ELEMS - 1) prefix[i / CHUNK_ELEMS] = j;\n        const unsigned char *e = src + i * (uint64_t)elem_size;\n        if (all_bytes_zero(e, elem_size)) {"),
    "float_compare_drops_negative_zero": ("if (p[b] != 0) return 0;", "if (p[b] != 0 && !(b == elem_size - 1 && p[b] == 0x80)) return 0;"),
    "decode_skips_counter": ("memcpy(e, val + j * (uint64_t)elem_size, (size_t)elem_size);\n            j += 1;\n        } else {\n            memset(e, 0, (size_t)elem_size);\n        }\n    }\n}\n\nvoid oracle_decompress_chunked",
                             "memcpy(e, val + j * (uint64_t)elem_size, (size_t)elem_size);\n            j += (i % 97 != 0);\n        } else {\n            memset(e, 0, (size_t)elem_size);\n        }\n    }\n}\n\nvoid oracle_decompress_chunked"),
    "relu_keeps_negatives": ("return f <= 0.0f; }\n    case ORACLE_F64", "return f == 0.0f; }\n    case ORACLE_F64"),
    "bwd_multiplies_instead_of_selecting": ("memset(o + i * (uint64_t)elem_size, 0, (size_t)elem_size);\n    }\n}\n\n/* M_b",
                                            "memmove(o + i * (uint64_t)elem_size, g + i * (uint64_t)elem_size, (size_t)elem_size);\n    }\n}\n\n/* M_b"),
    "prune_compare_not_strict": ("return f <= tau; }\n    case ORACLE_F64: { double d; memcpy(&d, e, 8); return d <= (double)tau; }",
                                 "return f < tau; }\n    case ORACLE_F64: { double d; memcpy(&d, e, 8); return d <= (double)tau; }"),
    "prune_by_magnitude": ("case ORACLE_F32: { float f; memcpy(&f, e, 4); return f <= tau; }",
                           "case ORACLE_F32: { float f; memcpy(&f, e, 4); return (f < 0 ? -f : f) <= tau; }"),
    "prune_drops_nan": ("case ORACLE_F32: { float f; memcpy(&f, e, 4); return f <= tau; }",
                        "case ORACLE_F32: { float f; memcpy(&f, e, 4); return !(f > tau); }"),
    "mask_drops_zero_values": ("if ((mask_bitmap[i >> 5] >> (i & 31)) & 1u) {\n            memcpy(val",
                               "if (((mask_bitmap[i >> 5] >> (i & 31)) & 1u) && !all_bytes_zero(e, elem_size)) {\n            memcpy(val"),
    "mask_msb_first": ("if ((mask_bitmap[i >> 5] >> (i & 31)) & 1u) {\n            memcpy(val",
                       "if ((mask_bitmap[i >> 5] >> (31 - (i & 31))) & 1u) {\n            memcpy(val"),
    "relu6_never_saturates": ("else if (ge6)         six_pattern(kind, act);", "else if (ge6 && 0)    six_pattern(kind, act);"),
    "relu6_bwd_passes_saturated_units": ("            pass = lt6;\n", "            pass = 1;\n"),
    "narrow_truncates_instead_of_rounding": ("if (rem > half || (rem == half && (q & 1u))) q += 1u;        /* a carry",
                                             "if (0) q += 1u;        /* a carry"),
    "narrow_half_ties_away_from_zero": ("if (rem > half || (rem == half && (q & 1u))) q += 1u;        /* a carry",
                                        "if (rem >= half) q += 1u;        /* a carry"),
    "narrow_bf16_ties_away_from_zero": ("if (rem > 0x8000u || (rem == 0x8000u && (q & 1u))) q += 1u;", "if (rem >= 0x8000u) q += 1u;"),
    "narrow_tests_zero_after_the_cast": ("        if (u != 0) {\n            values[j] = to_kind",
                                         "        if ((to_kind == ORACLE_F16 ? oracle_float_to_half(u) : oracle_float_to_bfloat16(u)) & 0x7FFFu) {\n            values[j] = to_kind"),
    "widen_bf16_shifts_one_bit_short": ("            } else {\n                u = (uint32_t)h << 16;", "            } else {\n                u = (uint32_t)h << 15;"),
    "widen_skips_the_value_counter": ("            uint16_t h = values[j];\n            j += 1;", "            uint16_t h = values[j];\n            j += (i % 89 != 0);"),
    "maxpool_last_of_equal_maxima_wins": ("if (k == 0 || v > best || v != v) {", "if (k == 0 || v >= best || v != v) {"),
    "maxpool_ignores_nan": ("if (k == 0 || v > best || v != v) {", "if (k == 0 || v > best) {"),
    "maxpool_codes_column_major": ("codes[o >> 4] |= (uint32_t)best_k << (2 * (o & 15));", "codes[o >> 4] |= (uint32_t)(((best_k & 1) << 1) | (best_k >> 1)) << (2 * (o & 15));"),
    "bytes_forgets_prefix": ("return 4 * words + nnz * (uint64_t)elem_size + 8 * chunks;", "return 4 * words + nnz * (uint64_t)elem_size;"),
    "bytes_counts_bits_as_bytes": ("return 4 * words + nnz", "return 32 * words + nnz"),
}


def build_mutant(tmp_path, name):
    old, new = MUTANTS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation site of {name} not found exactly once"
    c = tmp_path / f"{name}.c"
    c.write_text(text.replace(old, new))
    so = tmp_path / f"{name}.so"
    subprocess.check_call(["gcc", "-O1", "-std=c11", "-shared", "-fPIC", "-I", os.path.dirname(SRC), "-o", str(so), str(c)])
    L = ctypes.CDLL(str(so))
    u64, vp, i32 = ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int
    L.oracle_compress.restype = u64
    L.oracle_compress.argtypes = [vp, u64, i32, vp, vp, vp]
    L.oracle_decompress.argtypes = [vp, vp, u64, i32, vp]
    L.oracle_relu_fwd_compress.restype = u64
    L.oracle_relu_fwd_compress.argtypes = [vp, u64, i32, vp, vp, vp, vp]
    L.oracle_relu_bwd_from_bitmap.argtypes = [vp, vp, u64, i32, vp]
    L.oracle_prune_fwd_compress.restype = u64
    L.oracle_prune_fwd_compress.argtypes = [vp, u64, i32, ctypes.c_float, vp, vp, vp, vp]
    L.oracle_relu6_fwd_compress.restype = u64
    L.oracle_relu6_fwd_compress.argtypes = [vp, u64, i32, vp, vp, vp, vp]
    L.oracle_relu6_bwd_from_stash.argtypes = [vp, vp, u64, i32, vp, vp]
    L.oracle_mask_compress.restype = u64
    L.oracle_mask_compress.argtypes = [vp, u64, i32, vp, vp, vp]
    L.oracle_compressed_bytes.restype = u64
    L.oracle_compressed_bytes.argtypes = [u64, u64, i32]
    L.oracle_narrow_compress.restype = u64
    L.oracle_narrow_compress.argtypes = [vp, u64, i32, i32, ctypes.c_float, vp, vp, vp, vp]
    L.oracle_widen_decompress.restype = None
    L.oracle_widen_decompress.argtypes = [vp, vp, u64, i32, vp]
    L.oracle_maxpool2x2_fwd.restype = None
    L.oracle_maxpool2x2_fwd.argtypes = [vp, u64, u64, u64, i32, vp, vp]
    return L


def p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def pins_hold(L) -> bool:
    """A compact rerun of the independent pins against library `L`; False as soon as one fails."""
    n = 2 * 4096 + 77
    x = W.random_patterns(n, "f32", 0.5, seed=1)
    x[5] = 0x80000000                                             # a negative zero must survive
    nz = x != 0
    bitmap = np.zeros((n + 31) // 32, np.uint32)
    values = np.zeros(n, np.uint32)
    prefix = np.zeros((n + 4095) // 4096, np.uint64)
    nnz = L.oracle_compress(p(x), n, 4, p(bitmap), p(values), p(prefix))
    packed = np.packbits(nz, bitorder="little")
    ref_bitmap = np.concatenate([packed, np.zeros((-packed.size) % 4, np.uint8)]).view("<u4")
    per_chunk = np.add.reduceat(nz.astype(np.uint64), np.arange(0, n, 4096))
    ref_prefix = np.concatenate([[0], np.cumsum(per_chunk)[:-1]]).astype(np.uint64)
    if nnz != int(nz.sum()) or not np.array_equal(bitmap, ref_bitmap) or not np.array_equal(values[:nnz], x[nz]) \
            or not np.array_equal(prefix, ref_prefix):
        return False
    back = np.empty(n, np.uint32)
    L.oracle_decompress(p(bitmap), p(values), n, 4, p(back))
    if not np.array_equal(back, x):
        return False
    # ReLU pair against torch
    t = torch.randn(n, generator=torch.Generator().manual_seed(3)) * 2
    t[::53] = 0.0
    xr = W.raw_numpy(t)
    y = np.empty(n, np.uint32)
    L.oracle_relu_fwd_compress(p(xr), n, 0, p(y), p(bitmap), p(values), p(prefix))
    if not np.array_equal(y, W.raw_numpy(torch.relu(t) + 0.0)):
        return False
    g = torch.randn(n, generator=torch.Generator().manual_seed(4))
    gin = np.empty(n, np.uint32)
    L.oracle_relu_bwd_from_bitmap(p(bitmap), p(W.raw_numpy(g)), n, 4, p(gin))
    if not np.array_equal(gin, W.raw_numpy(torch.where(t > 0, g, torch.zeros(())))):
        return False
    # pruning: torch.where on a tensor with close-to-zero values of both signs, the threshold itself and a NaN
    tp = torch.randn(n, generator=torch.Generator().manual_seed(5)) * 0.08
    tp[:4] = torch.tensor([0.05, float("nan"), -0.2, 0.0])
    tau = torch.tensor(0.05, dtype=torch.float32)
    yp = np.empty(n, np.uint32)
    L.oracle_prune_fwd_compress(p(W.raw_numpy(tp)), n, 0, ctypes.c_float(0.05), p(yp), p(bitmap), p(values), p(prefix))
    if not np.array_equal(yp, W.raw_numpy(torch.where(tp <= tau, torch.zeros(()), tp))):
        return False
    # double mask: numpy boolean indexing under a mask that also covers zero elements
    rng = np.random.default_rng(9)
    mask = rng.random(n) < 0.4
    mp = np.packbits(mask, bitorder="little")
    mbm = np.concatenate([mp, np.zeros((-mp.size) % 4, np.uint8)]).view("<u4").copy()
    ym = np.empty(n, np.uint32)
    vm = np.zeros(n, np.uint32)
    cnt = L.oracle_mask_compress(p(x), n, 4, p(mbm), p(ym), p(vm))
    if cnt != int(mask.sum()) or not np.array_equal(vm[:cnt], x[mask]) or not np.array_equal(ym, np.where(mask, x, 0)):
        return False
    # ReLU6 pair against torch
    t6 = torch.randn(n, generator=torch.Generator().manual_seed(6)) * 4
    t6[:3] = torch.tensor([6.0, 7.5, 0.0])
    y6 = np.empty(n, np.uint32)
    nnz6 = L.oracle_relu6_fwd_compress(p(W.raw_numpy(t6)), n, 0, p(y6), p(bitmap), p(values), p(prefix))
    if not np.array_equal(y6, W.raw_numpy(torch.nn.functional.relu6(t6) + 0.0)):
        return False
    g6 = torch.randn(n, generator=torch.Generator().manual_seed(7))
    gin6 = np.empty(n, np.uint32)
    L.oracle_relu6_bwd_from_stash(p(bitmap), p(values[:nnz6].copy()), n, 0, p(W.raw_numpy(g6)), p(gin6))
    if not np.array_equal(gin6, W.raw_numpy(torch.where((t6 > 0) & (t6 < 6), g6, torch.zeros(())))):
        return False
    # down-cast on stash against numpy (binary16) and torch (bfloat16), with ties and an underflow
    tn = torch.randn(n, generator=torch.Generator().manual_seed(8))
    xn = W.raw_numpy(tn).copy()
    xn[:6] = np.array([0x3F801000, 0x3F803000, 0x3F808000, 0x3F818000, 0x2F000000, 0], dtype=np.uint32)
    for to_kind, ref in ((1, xn.view(np.float32).astype(np.float16).view(np.uint16)),
                         (2, torch.from_numpy(xn.view(np.int32)).view(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))):
        v16 = np.zeros(n, np.uint16)
        nn_ = L.oracle_narrow_compress(p(xn), n, to_kind, 0, 0.0, None, p(bitmap), p(v16), p(prefix))
        if nn_ != int(np.count_nonzero(xn)) or not np.array_equal(v16[:nn_], ref[xn != 0]):
            return False
        # and back up: the narrowed dense tensor cast to binary32 by the library (exact)
        wide = np.empty(n, np.uint32)
        L.oracle_widen_decompress(p(bitmap), p(v16), n, to_kind, p(wide))
        dense16 = np.where(xn != 0, ref, 0).astype(np.uint16)
        up = dense16.view(np.float16).astype(np.float32).view(np.uint32) if to_kind == 1 else dense16.astype(np.uint32) << 16
        if not np.array_equal(wide, up):
            return False
    # 2x2 max pooling against torch: values and winner positions, with ties and a NaN
    tp = torch.clamp_min(torch.randn(3, 8, 12, generator=torch.Generator().manual_seed(9)), 0.0)
    tp[0, 0, 1] = float("nan"); tp[0, 3, 2] = float("nan"); tp[1, 2:4, 2:4] = 1.5
    yp = np.empty(3 * 4 * 6, np.uint32)
    cp = np.zeros((3 * 4 * 6 + 15) // 16, np.uint32)
    L.oracle_maxpool2x2_fwd(p(W.raw_numpy(tp.reshape(-1))), 3, 8, 12, 0, p(yp), p(cp))
    refp, idxp = torch.nn.functional.max_pool2d(tp.unsqueeze(0), 2, return_indices=True)
    kk = (2 * (idxp[0] // 12 - 2 * torch.arange(4).view(1, 4, 1)) + (idxp[0] % 12 - 2 * torch.arange(6).view(1, 1, 6))).reshape(-1).numpy()
    unpacked = (cp.repeat(16) >> np.tile(2 * np.arange(16, dtype=np.uint32), cp.size)) & 3
    if not np.array_equal(unpacked[:kk.size], kk.astype(np.uint32)):
        return False
    if not np.array_equal(np.nan_to_num(yp.view(np.float32), nan=9.0), np.nan_to_num(refp.reshape(-1).numpy(), nan=9.0)):
        return False
    # closed form and the first row of Table 1 (16,3,224,224 at 50 % non-zero: 4.88 MB without the prefix term)
    if L.oracle_compressed_bytes(200704, 100352, 4) != 200704 // 8 + 4 * 100352 + 8 * 49:
        return False
    mb = (L.oracle_compressed_bytes(2408448, 1204224, 4) - 8 * (2408448 // 4096)) / 2 ** 20
    return abs(mb - 4.88) <= 0.005


def test_the_unmutated_source_passes(tmp_path):
    MUTANTS["identity"] = ("#define CHUNK_ELEMS 4096u", "#define CHUNK_ELEMS 4096u")
    try:
        assert pins_hold(build_mutant(tmp_path, "identity"))
    finally:
        del MUTANTS["identity"]


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_every_planted_mistake_is_caught(tmp_path, name):
    assert not pins_hold(build_mutant(tmp_path, name)), f"the pins did not notice: {name}"
