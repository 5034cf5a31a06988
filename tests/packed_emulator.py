"""numpy walk over a packed layer that follows the documented item/table addressing of the CUDA
kernel (paper_2608_15602_b200/csrc/fluxbin_layout.h) step by step.  Host-logic test helper: it
lets the CPU suite check the packer's layout against the oracle without a GPU."""
import struct

import numpy as np

HEADER_FMT = "<II20i7Q"


def parse_header(buf):
    f = struct.unpack_from(HEADER_FMT, buf.tobytes()[:256])
    names = ["magic", "version", "M", "N", "Kb", "Ks", "g", "n_sal", "Mpad", "nrb", "sps0", "sps1", "nunits0",
             "nunits1", "npairs0", "npairs1", "item_bytes0", "item_bytes1", "n_sal_svec", "n_dead", "sal_last_w", "reserved0",
             "off_coldesc", "off_items0", "off_items1", "off_sal_idx", "off_dead_ids", "off_dead_scales",
             "total_bytes"]
    return dict(zip(names, f))


def _f16(u16):
    return np.asarray(u16, np.uint16).view(np.float16).astype(np.float64)


def emulate_linear(buf, x_bits):
    """y[B][M] in fp64 from the packed bytes and fp16 activations x_bits [B][>=N]."""
    h = parse_header(buf)
    xs = _f16(x_bits)
    B = xs.shape[0]
    y = np.zeros((B, h["Mpad"]))
    signs = np.array([[1.0 if (p >> n) & 1 else -1.0 for n in range(8)] for p in range(256)])   # [256][8]
    lanes = np.arange(32)
    for region in (0, 1):
        npairs, sps, ib_full = h[f"npairs{region}"], h[f"sps{region}"], h[f"item_bytes{region}"]
        for P in range(npairs):
            # the last salient pair may be narrow: w = 8 or 16 steps per item instead of 32 (all 32 table slots
            # are still built; the column table repeats the live ones)
            w = h["sal_last_w"] if (region == 1 and sps == 1 and P == npairs - 1) else 32
            ib = ib_full if w == 32 else 96 * w
            nseg = w // sps
            off = h["off_coldesc"] + ((h["npairs0"] if region else 0) + P) * 1024
            cd = buf[off:off + 1024].view(np.uint16).reshape(32, 8, 2)
            a = xs[:, cd[:, :, 0].astype(np.int64)] * _f16(cd[:, :, 1])[None]      # [B][32][8]
            tables = np.einsum("bsn,pn->bsp", a, signs)                              # [B][32][256]
            for rb in range(h["nrb"]):
                ioff = h[f"off_items{region}"] + P * h["nrb"] * ib_full + rb * ib
                item = buf[ioff:ioff + ib]
                sc = item[32 * w:].view(np.uint16)
                for s in range(w):
                    sigma = lanes ^ s
                    if w == 32:
                        byte = item[(s >> 4) * 512 + lanes * 16 + (s & 15)].astype(np.int64)
                    else:
                        byte = item[lanes * w + s].astype(np.int64)
                    j = s // sps
                    if nseg <= 8:
                        scale = _f16(sc[lanes * nseg + j])
                    else:
                        scale = _f16(sc[(j >> 3) * 256 + lanes * 8 + (j & 7)])
                    y[:, rb * 32 + lanes] += scale[None] * tables[:, sigma, byte]
    return y[:, :h["M"]]
