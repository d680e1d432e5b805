"""Writes q4nx_k32_n32.hex: the 640-byte Q4NX container of a 32 x 32 matrix, by hand rule.

The file is an INPUT fixture for the layout tests; its content follows directly from the layout
statement (block = codes, scales, offsets; code line r = row r, low nibble first) and the matrix
code[n][k] = (k + 3n) mod 16, scale 0.5, offset -1.  No library or oracle code is involved.
"""
import os

lines = ["# Q4NX container of the 32 x 32 matrix code[n][k] = (k + 3n) mod 16, scale 0.5, offset -1.",
         "# One tail block with a single 32-group: 512 code bytes, 64 scale bytes, 64 offset bytes = 640.",
         "# Layout reading of Sec. 'Dequantization Engine' (block = codes, then scales, then offsets);",
         "# code line r = row r of the strip, 16 bytes, byte p = code[2p] | code[2p+1] << 4."]
for r in range(32):
    row = ["%02x" % (((2 * p + 3 * r) % 16) | (((2 * p + 1 + 3 * r) % 16) << 4)) for p in range(16)]
    lines.append(" ".join(row) + "   # codes row %d" % r)
for i in range(4):
    lines.append(" ".join(["00 3f"] * 8) + "   # scales rows %d..%d = 0.5 (bf16 0x3f00, little-endian)" % (8 * i, 8 * i + 7))
for i in range(4):
    lines.append(" ".join(["80 bf"] * 8) + "   # offsets rows %d..%d = -1 (bf16 0xbf80)" % (8 * i, 8 * i + 7))
with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "q4nx_k32_n32.hex"), "w") as f:
    f.write("\n".join(lines) + "\n")
