"""Oracle (test infrastructure, not part of the product) for the re-encoding of MX4 / MX6 operands onto
the 8-bit block-scaled tensor format: E4M3 element bytes plus one power-of-two scale byte per 32 elements.

The paper has no counterpart; the definition followed here is the one the library documents for
bdr_reencode_e4m3 (include/bdr.h):
  * the operand is quantized as in Section III (the oracle's own encode / quant_dequant);
  * two neighbouring 16-element blocks with exponent fields F0, F1 form a group with S = max(F0, F1); the
    group's scale byte is S - 7 (scale 2^(S-7-127)) when 16 <= S < 255, else 0;
  * an element's byte is the E4M3 code (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, gradual
    underflow, no infinities) of value / scale, sign of zero kept;
  * `inexact` is raised when a value / scale is not an E4M3 number, when a block with F < 16 holds a
    non-zero magnitude, or when a block has F = 255; the bytes are then unspecified.
Plain numpy, one step after the other; pinned in tests/test_oracle_pins.py (byte encoder against a
library cast, representability limits, value reconstruction)."""
import numpy as np

from oracle import oracle as orc


def e4m3_value_table() -> np.ndarray:
    """The 128 non-negative E4M3 codes as float64 (code 0x7F, the NaN, as nan)."""
    v = np.empty(128, dtype=np.float64)
    for code in range(128):
        e, man = code >> 3, code & 7
        v[code] = man * 2.0 ** -9 if e == 0 else (1.0 + man / 8.0) * 2.0 ** (e - 7)
    v[0x7F] = np.nan
    return v


def e4m3_bytes(values: np.ndarray):
    """(bytes, representable): the E4M3 byte of every value that is an E4M3 number (0 elsewhere)."""
    table = e4m3_value_table()
    mag = np.abs(values.astype(np.float64))
    order = np.argsort(table[:0x7F])                      # finite codes, ascending values (already sorted)
    idx = np.searchsorted(table[:0x7F][order], mag)
    idx = np.minimum(idx, 0x7E)
    hit = table[idx] == mag
    out = np.where(hit, idx, 0).astype(np.uint8)
    out |= (np.signbit(values).astype(np.uint8) << 7)
    return out, hit


def reencode_e4m3(cfg: orc.Config, x: np.ndarray):
    """x [rows, K] fp32 (rows % 128 == 0, K % 128 == 0) -> (bytes [rows, K] u8, scales u8 in atom order, inexact)."""
    assert cfg.k1 == 16 and cfg.k2 == 2 and cfg.d2 == 1 and cfg.m in (2, 4)
    rows, K = x.shape
    assert rows % 128 == 0 and K % 128 == 0
    y, _ = orc.quant_dequant(cfg, x)
    F, _, code = orc.encode(cfg, x)
    F = F.astype(np.int64)
    nonzero_block = ((code & ((1 << cfg.m) - 1)) != 0).reshape(rows, K // 16, 16).any(axis=2)
    S = F.reshape(rows, K // 32, 2).max(axis=2)
    in_range = (S >= 16) & (S < 255)
    sb = np.where(in_range, S - 7, 0)
    scale = np.ldexp(1.0, sb - 127)
    v = y.astype(np.float64) / np.repeat(scale, 32, axis=1)
    with np.errstate(invalid="ignore"):
        out, hit = e4m3_bytes(np.where(np.isfinite(v), v, 0.0))
    inexact = bool((~hit).any() or (nonzero_block & (F < 16)).any() or (F == 255).any())
    # scale bytes: atom [K chunk of 128][row tile of 128], byte (r % 32) * 16 + ((r % 128) // 32) * 4 + group % 4
    atoms = sb.astype(np.uint8).reshape(rows // 128, 4, 32, K // 128, 4)   # [tile][r // 32][r % 32][chunk][g % 4]
    scales = np.ascontiguousarray(atoms.transpose(3, 0, 2, 1, 4)).reshape(-1)
    return out, scales, inexact
