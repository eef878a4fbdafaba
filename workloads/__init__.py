"""Seeded synthetic inputs (shared by tests, benchmark and smoke check; no method arithmetic)."""
